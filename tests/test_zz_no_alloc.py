"""The entry point for callers that cannot allocate device memory
(``baps_attention_restart_rates_static``) against the ordinary one
(``baps_attention_restart_rates``), through the C ABI.

Such callers -- plug-ins working inside a fixed memory budget set by their host application,
serving loops where an allocation would stall the device, processes whose allocator belongs to
another framework -- hand in inputs and outputs only; the per-query-tile counters live in an array
built into the library.  The file is named so that pytest collects it last.
"""
import pytest
import torch

from paper_2602_02071_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def _case(seed, S, lam):
    w = workloads.AttnWorkload("t", 1, 4, 2, S, 128, True, 128, 128, outlier_frac=0.01, seed=seed)
    q, k, v = workloads.make_qkv(w, device="cuda")
    out_ref, rates_ref = binding.baps_attention_restart_rates(q, k, v, causal=True, lam=lam)
    out = torch.empty_like(q)
    rates = torch.full((2,), -1.0, dtype=torch.float32, device="cuda")
    binding.baps_attention_restart_rates_static(q, k, v, causal=True, out=out, rates=rates, lam=lam)
    binding.poll_async_error()
    # same kernels, same inputs: the rates are ratios of identical integer counts, the output is
    # the same bf16 tensor
    assert torch.equal(rates, rates_ref), (rates.tolist(), rates_ref.tolist())
    assert torch.equal(out, out_ref)
    assert float(rates_ref[0]) > 0.0          # the outlier keys do force restarts


def test_static_scratch_matches_caller_scratch_twice_in_a_row():
    # two calls in a row: a larger problem first, then a smaller one with another lambda, so that
    # counters left behind by the first call would show up in the second if they were read
    _case(seed=31, S=2048, lam=1)
    _case(seed=32, S=1024, lam=0)


def test_static_scratch_limit_is_enforced():
    lib = binding.load()
    assert binding.status_string(-6).startswith("BAPS_ERR_SCRATCH_LIMIT")
    # B * H * S / 128 = 64 * 64 * 128 = 524288 counters > 262144: refused before anything is launched
    n = 64 * 64 * 16384 * 128
    q = torch.empty(1, dtype=torch.bfloat16, device="cuda")      # never dereferenced
    rates = torch.empty(2, dtype=torch.float32, device="cuda")
    rc = lib.baps_attention_restart_rates_static(q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr(),
                                                 64, 64, 64, 16384, 128, 1, 128, 128, 1, rates.data_ptr(), None)
    assert rc == -6 and n > 0
