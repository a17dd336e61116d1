"""GPU parity: the CUDA-core float32 attention kernel against the CPU checker."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_02071_b200 import binding, workloads
from parity import gate_attention

pytestmark = pytest.mark.gpu


def _run(w, lam=1, mode=binding.MODE_E2E_HIF8, b0_last=False):
    q, k, v = workloads.make_qkv(w)
    st = binding.baps_attention_fwd_ex(q.cuda(), k.cuda(), v.cuda(), causal=w.causal,
                                       block_q=w.block_q, block_k=w.block_k, lam=lam, mode=mode, b0_last=b0_last)
    torch.cuda.synchronize()
    ref = oracle.attention(q.numpy(), k.numpy(), v.numpy(), causal=w.causal, block_q=w.block_q,
                           block_k=w.block_k, lam=lam, b0_last=b0_last,
                           mode={binding.MODE_EXACT: oracle.MODE_EXACT, binding.MODE_E2E_HIF8: oracle.MODE_E2E_HIF8,
                                 binding.MODE_EXP2_HIF8: oracle.MODE_EXP2_HIF8}[mode])
    return st, ref


def test_config1_single_head():
    w = workloads.WORKLOADS["c1_single_head"]
    st, ref = _run(w)
    info = gate_attention(st.out_f32.cpu().numpy(), ref, what="c1")
    assert np.array_equal(st.row_m.cpu().numpy().reshape(ref.row_m.shape), ref.row_m)
    assert np.array_equal(st.restarts.cpu().numpy().ravel(), ref.restarts)
    assert np.allclose(st.row_d.cpu().numpy().reshape(ref.row_d.shape), ref.row_d, rtol=1e-5)
    # plain entry point gives the same numbers
    q, k, v = workloads.make_qkv(w)
    out = binding.baps_attention_fwd_f32(q.cuda(), k.cuda(), v.cuda(), causal=False, block_q=64, block_k=64)
    assert torch.equal(out, st.out_f32)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("bq", [64, 128])
@pytest.mark.parametrize("lam", [0, 1, 2])
def test_f32_kernel_shapes(causal, bq, lam):
    w = workloads.AttnWorkload("t", 2, 4, 2, 512, 64 if bq == 64 else 128, causal, bq, bq, dtype="f32", seed=bq + lam)
    st, ref = _run(w, lam=lam)
    gate_attention(st.out_f32.cpu().numpy(), ref, what=f"f32 causal={causal} bq={bq} lam={lam}")
    assert np.array_equal(st.restarts.cpu().numpy().ravel(), ref.restarts)


def test_f32_kernel_outliers_and_exact_mode():
    w = workloads.AttnWorkload("t", 1, 2, 2, 1024, 128, True, 128, 128, dtype="f32", outlier_frac=0.01, seed=4)
    st, ref = _run(w)
    gate_attention(st.out_f32.cpu().numpy(), ref, what="f32 outliers")
    st, ref = _run(w, mode=binding.MODE_EXACT)
    err = np.abs(st.out_f32.cpu().numpy().reshape(ref.out.shape) - ref.out)
    assert err.max() < 1e-4


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("bq", [64, 128])
def test_f32_kernel_exp2_setup(causal, bq):
    """The "Exp2 HiF8" setup of Section 4.1 on the CUDA cores."""
    w = workloads.AttnWorkload("t", 1, 4, 2, 512, 64 if bq == 64 else 128, causal, bq, bq, dtype="f32",
                               outlier_frac=0.01, seed=60 + bq)
    st, ref = _run(w, mode=binding.MODE_EXP2_HIF8)
    gate_attention(st.out_f32.cpu().numpy(), ref, what=f"f32 exp2 causal={causal} bq={bq}")
    assert np.allclose(st.row_m.cpu().numpy().reshape(ref.row_m.shape), ref.row_m, rtol=1e-5, atol=1e-5)
    assert int(st.restarts.sum()) == 0


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("bq,S", [(64, 64), (64, 512), (128, 256)])
def test_f32_kernel_b0_first_and_last(causal, bq, S):
    """B0 = {first, last visible key tile} on the CUDA cores (order 0, last, 1, ..., last - 1)."""
    w = workloads.AttnWorkload("t", 1, 4, 2, S, 64 if bq == 64 else 128, causal, bq, bq, dtype="f32",
                               outlier_frac=0.02, seed=80 + bq + S)
    st, ref = _run(w, b0_last=True)
    gate_attention(st.out_f32.cpu().numpy(), ref, what=f"f32 b0 first+last causal={causal} bq={bq} S={S}")
    assert np.array_equal(st.restarts.cpu().numpy().ravel(), ref.restarts)
