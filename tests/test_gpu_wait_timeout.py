"""A bounded device-side wait that runs out is reported through baps_poll_async_error() and leaves
the library usable.

No fault, trap or endless loop is involved: a second build of the library (``libbaps_waittest.so``:
same sources, every wait limited to 1 ms, plus a test-only switch) lets the TMA producer of the
fused kernel leave out one key-tile load on a one-CTA problem.  The MMA role waits for that tile,
gives up after its limit and raises the CTA's abort flag; the softmax warps run through the rest of
their task list with every wait returning at once, all roles meet at the common teardown, tensor
memory is released and the kernel returns.  The host then reads the status.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2602_02071_b200 import binding, build, workloads

pytestmark = pytest.mark.gpu

TIMEOUT, OK = -5, 0


@pytest.fixture(scope="module")
def wlib():
    lib = ctypes.CDLL(build.build_wait_test())
    vp, i = ctypes.c_void_p, ctypes.c_int
    lib.baps_attention_fwd.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, i, vp]
    lib.baps_attention_restart_rates.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, i, i, vp, ctypes.c_size_t, vp, vp]
    lib.baps_poll_async_error.argtypes = [vp]
    lib.baps_test_skip_kv_load.argtypes = [i]
    return lib


def _fwd(lib, w, q, k, v, out):
    return lib.baps_attention_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), w.B, w.H, w.Hkv, w.S,
                                  w.D, int(w.causal), 128, 128, None)


def test_expired_wait_is_reported_once_and_the_next_launch_is_correct(wlib):
    # one CTA: one head, two query tiles, two key tiles (four tile loads: K_0, V_0, K_1, V_1)
    w = workloads.AttnWorkload("t", 1, 1, 1, 256, 128, False, 128, 128, seed=77)
    q, k, v = workloads.make_qkv(w, device="cuda")
    out = torch.zeros_like(q)
    assert wlib.baps_poll_async_error(None) == OK
    assert wlib.baps_test_skip_kv_load(2) == 0                    # K_1 never arrives
    assert _fwd(wlib, w, q, k, v, out) == OK                       # launch errors only: the call is asynchronous
    assert wlib.baps_poll_async_error(None) == TIMEOUT
    assert wlib.baps_poll_async_error(None) == OK                  # the record is cleared by the first poll
    assert not out.any()                                           # nothing was stored after the abort
    # restart rates of a call whose wait expired are NaN, not numbers made from stale counters
    scratch = torch.full((2,), 7, dtype=torch.int32, device="cuda")
    rates = torch.zeros(2, dtype=torch.float32, device="cuda")
    assert wlib.baps_attention_restart_rates(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), 1, 1, 1, 256,
                                             128, 0, 128, 128, 1, scratch.data_ptr(), 2, rates.data_ptr(), None) == OK
    torch.cuda.synchronize()
    assert torch.isnan(rates).all()
    assert wlib.baps_poll_async_error(None) == TIMEOUT
    # switch the omission off: the same library, same context, now gives the right answer
    assert wlib.baps_test_skip_kv_load(-1) == 0
    assert _fwd(wlib, w, q, k, v, out) == OK
    assert wlib.baps_poll_async_error(None) == OK
    assert torch.equal(out, binding.baps_attention_fwd(q, k, v, causal=False))
    ref = oracle.attention(q.float().cpu().numpy(), k.float().cpu().numpy(), v.float().cpu().numpy(), causal=False,
                           block_q=128, block_k=128)
    got = out.float().cpu().numpy().reshape(ref.out.shape)
    assert np.abs(got - ref.out).max() <= 1e-2 + 2.0 ** -7 * np.abs(ref.out).max()   # bf16 output
