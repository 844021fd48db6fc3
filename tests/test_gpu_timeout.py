"""The give-up path of the bounded on-chip waits, exercised without faulting anything.

Every wait in the kernels has a time limit.  With the diagnostic limit of one nanosecond the first
wait that is not already satisfied runs out: the kernel must raise ADWIN_DEV_TIMEOUT, let its own
copies land, free its tensor memory and return -- and the very next ordinary call on the same
inputs must match the oracle, which shows that the context and the device state are intact.
"""
import numpy as np
import pytest
import torch

from paper_2605_28396_b200 import api, synth
from tests import test_gpu_lmhead as L
from tests import test_gpu_parity as G

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture()
def one_nanosecond_limit():
    api.adwin_diag_set_wait_limit_ns(1)
    try:
        yield
    finally:
        api.adwin_diag_set_wait_limit_ns(0)


def test_staged_kernel_gives_up_cleanly(one_nanosecond_limit):
    batch = synth.make_batch(1, device=DEV, B=1, T=6, V=4096)
    batch.window = torch.tensor([6], dtype=torch.int32, device=DEV)
    grad = torch.zeros(batch.shape, dtype=torch.float32, device=DEV)
    out = api.adwin_opd_kl_fwd_bwd(batch.student, batch.teacher, batch.tokens, batch.window,
                                   batch.rollout_len, grad=grad, flags=api.FORCE_STAGED)
    torch.cuda.synchronize()
    assert int(out.dev_status.item()) & api.DEV_TIMEOUT
    api.adwin_diag_set_wait_limit_ns(0)
    G.run_and_check(batch, grad_dtype=torch.float32, flags=api.FORCE_STAGED)


def test_tensor_core_kernels_give_up_cleanly(one_nanosecond_limit):
    batch = synth.make_lmhead_batch(DEV, B=1, T=130, V=512, d_s=64, d_t=64, w_std=0.1)
    batch.window[:] = 130
    dW = torch.zeros((512, 64), dtype=torch.float32, device=DEV)
    out = api.adwin_opd_kl_lmhead_fwd_bwd(batch.hidden_student, batch.w_student,
                                          batch.hidden_teacher, batch.w_teacher, batch.tokens,
                                          batch.window, batch.rollout_len, grad_w=dW)
    torch.cuda.synchronize()
    assert int(out.dev_status.item()) & api.DEV_TIMEOUT
    api.adwin_diag_set_wait_limit_ns(0)
    got = L.run(batch)
    L.check_all(batch, got, L.oracle(batch, api.GRAD_FULL_KL, 0), 0)
