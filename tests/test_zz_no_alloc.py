"""The entry point that allocates nothing, against the ordinary one (collected last on purpose).

Some users of the library hold all of their device memory before the first call and cannot
allocate afterwards (a framework-owned memory pool, a latency-critical loop).  For them
``adwin_opd_kl_fwd_bwd_no_alloc`` keeps its row map in a fixed array inside the library.  This test
calls it twice in a row through the C ABI, with different windows, shapes and gradient modes, so
that a second call that reused anything the first one left in that array would be caught, and
compares every output with ``adwin_opd_kl_fwd_bwd`` on the same inputs.
"""
import gc

import pytest
import torch

from paper_2605_28396_b200 import api, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _both(batch, mode, flags, grad_dtype):
    B, T, V = batch.shape
    f32 = dict(dtype=torch.float32, device=DEV)
    ref_grad = torch.full((B, T, V), 3.0, dtype=grad_dtype, device=DEV)
    ref = api.adwin_opd_kl_fwd_bwd(batch.student, batch.teacher, batch.tokens, batch.window,
                                   batch.rollout_len, grad=ref_grad, grad_mode=mode, flags=flags,
                                   grad_scale=0.5)
    # every buffer of the no-allocation call exists before the call
    grad = torch.full((B, T, V), 3.0, dtype=grad_dtype, device=DEV)
    kl, c, q = (torch.full((B, T), -1.0, **f32) for _ in range(3))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    gc.collect()   # tensors that earlier tests left in reference cycles must not be freed midway
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated(DEV)
    api.adwin_opd_kl_fwd_bwd_no_alloc(batch.student, batch.teacher, batch.tokens, batch.window,
                                      batch.rollout_len, grad=grad, kl=kl, logratio=c, gsq=q,
                                      dev_status=status, grad_mode=mode, flags=flags,
                                      grad_scale=0.5)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated(DEV) == before
    assert int(status.item()) == 0 and int(ref.dev_status.item()) == 0
    # same kernels on the same values: the tolerances of the host-buffer comparison apply
    assert torch.allclose(kl, ref.kl, rtol=1e-6, atol=1e-7)
    assert torch.allclose(c, ref.logratio, rtol=1e-6, atol=1e-7)
    assert torch.allclose(q, ref.gsq, rtol=1e-5, atol=1e-12)
    assert torch.equal(grad, ref_grad)


def test_no_alloc_entry_point_matches_on_two_calls_in_a_row():
    assert api.adwin_no_alloc_max_sequences() >= 1024
    first = synth.make_batch(2, device=DEV, B=5, T=24, V=8192, ragged_rollout=True)
    first.window = torch.tensor([24, 3, 0, 17, 9], dtype=torch.int32, device=DEV)
    _both(first, api.GRAD_FULL_KL, api.ZERO_TAIL, torch.bfloat16)
    second = synth.make_batch(3, device=DEV, B=2, T=10, V=151936)
    second.window = torch.tensor([4, 10], dtype=torch.int32, device=DEV)
    _both(second, api.GRAD_SAMPLED, api.RANGE_FULL, torch.float32)


def test_no_alloc_entry_point_rejects_batches_beyond_its_array():
    B = api.adwin_no_alloc_max_sequences() + 1
    z = torch.zeros((B, 1, 8), dtype=torch.bfloat16, device=DEV)
    i32 = dict(dtype=torch.int32, device=DEV)
    one = torch.zeros((B, 1), dtype=torch.float32, device=DEV)
    with pytest.raises(api.AdwinError) as e:
        api.adwin_opd_kl_fwd_bwd_no_alloc(z, z, torch.zeros((B, 1), **i32), torch.ones(B, **i32),
                                          None, grad=None, kl=one, logratio=one, gsq=None,
                                          dev_status=torch.zeros(1, **i32))
    assert e.value.code == 6
