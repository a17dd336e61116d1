"""GPU parity: the tensor-core BAPS attention kernel against the CPU checker.

Small problems are compared on every query tile; the benchmark configurations at full size on
a fixed sample of query tiles (first, second, middle, last of several heads, plus random ones),
which the checker computes one by one.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_02071_b200 import binding, workloads
from parity import EPS_REL, gate_attention

pytestmark = pytest.mark.gpu


def _run_gpu(w, q, k, v, lam=1, mode=binding.MODE_E2E_HIF8, b0_last=False):
    st = binding.baps_attention_fwd_ex(q, k, v, causal=w.causal, block_q=128, block_k=128, lam=lam, mode=mode,
                                       b0_last=b0_last)
    binding.poll_async_error()
    return st


def _np(t):
    return t.float().cpu().numpy()


def _select(arr, tiles, bq=128):
    """arr: [B,H,S,...] numpy; returns [n_sel, bq, ...]"""
    return np.stack([arr[b, h, i * bq:(i + 1) * bq] for b, h, i in tiles])


def _check(w, tiles=None, lam=1, what="", mode=binding.MODE_E2E_HIF8, b0_last=False):
    q, k, v = workloads.make_qkv(w)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    st = _run_gpu(w, qd, kd, vd, lam=lam, mode=mode, b0_last=b0_last)
    if tiles is None:
        tiles = [tuple(x) for x in oracle.all_tiles(w.B, w.H, w.S, 128)]
    assert mode in (binding.MODE_E2E_HIF8, binding.MODE_EXP2_HIF8)
    ref = oracle.attention(_np(q), _np(k), _np(v), causal=w.causal, block_q=128, block_k=128, lam=lam,
                           tiles=np.array(tiles, dtype=np.int32), b0_last=b0_last,
                           mode=oracle.MODE_E2E_HIF8 if mode == binding.MODE_E2E_HIF8 else oracle.MODE_EXP2_HIF8)
    got = _select(st.out_f32.cpu().numpy(), tiles)
    info = gate_attention(got, ref, what=what or w.name)
    # bookkeeping: the max (an integer in Algorithm 1, bit for bit; real valued in the Exp2 setup) and
    # the restart counts agree wherever no decision sat on a boundary
    clear = ref.row_margin >= EPS_REL
    gm = _select(st.row_m.cpu().numpy()[..., None], tiles)[..., 0]
    if mode == binding.MODE_E2E_HIF8:
        assert np.array_equal(gm[clear], ref.row_m[clear]), what
    else:
        assert np.allclose(gm, ref.row_m, rtol=1e-5, atol=1e-5), what
    gd = _select(st.row_d.cpu().numpy()[..., None], tiles)[..., 0]
    assert np.allclose(gd[clear], ref.row_d[clear], rtol=2e-2), what
    tile_clear = clear.all(axis=1)
    gr = np.array([st.restarts.cpu().numpy()[b, h, i] for b, h, i in tiles])
    assert np.array_equal(gr[tile_clear], ref.restarts[tile_clear]), what
    # bf16 output is the rounding of the fp32 one
    ob = _select(st.out.float().cpu().numpy(), tiles)
    assert np.abs(ob - got).max() <= np.abs(got).max() * 2.0 ** -8
    return info, st, (qd, kd, vd)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("D", [128, 64])
@pytest.mark.parametrize("S", [128, 384, 1024])
def test_small_problems_all_tiles(causal, D, S):
    w = workloads.AttnWorkload("t", 2, 4, 2, S, D, causal, 128, 128, seed=S + D + causal)
    _check(w, what=f"S={S} D={D} causal={causal}")


@pytest.mark.parametrize("B,H,Hkv,S,D,causal", [(3, 6, 2, 128, 128, True), (1, 3, 3, 256, 64, False),
                                               (2, 6, 2, 640, 64, True), (1, 12, 4, 896, 128, False)])
def test_unusual_shapes(B, H, Hkv, S, D, causal):
    """Single-tile sequences, an odd number of query tiles, three query heads per kv head."""
    w = workloads.AttnWorkload("t", B, H, Hkv, S, D, causal, 128, 128, outlier_frac=0.01, seed=B + H + S)
    _check(w, what=f"B{B} H{H} Hkv{Hkv} S{S} D{D} causal={causal}")
    _check(w, what="exp2", mode=binding.MODE_EXP2_HIF8)


@pytest.mark.parametrize("lam", [0, 2, 3])
def test_lambda_values(lam):
    w = workloads.AttnWorkload("t", 1, 4, 4, 768, 128, True, 128, 128, seed=lam)
    _check(w, lam=lam, what=f"lambda={lam}")


def test_outliers_force_restarts_and_general_path():
    w = workloads.AttnWorkload("t", 1, 4, 2, 1024, 128, True, 128, 128, outlier_frac=0.01, seed=5)
    info, st, _ = _check(w, what="outliers")
    assert int(st.restarts.sum()) > 0


def test_key_bias_non_causal_d64():
    w = workloads.AttnWorkload("t", 2, 4, 4, 1024, 64, False, 128, 128, key_bias_var=0.5, seed=6)
    _check(w, what="vit-like")


def test_matches_cuda_core_kernel_and_plain_entry_point():
    """Same inputs through the CUDA-core fp32 kernel (double-precision scores) and through the
    plain bf16 entry point."""
    w = workloads.AttnWorkload("t", 1, 2, 1, 512, 128, True, 128, 128, seed=8)
    q, k, v = workloads.make_qkv(w, device="cuda")
    st = _run_gpu(w, q, k, v)
    st32 = binding.baps_attention_fwd_ex(q.float(), k.float(), v.float(), causal=True, block_q=128, block_k=128)
    err = (st.out_f32 - st32.out_f32).abs()
    assert float(err.mean()) < 1e-3 and float(err.max()) < 5e-2
    out = binding.baps_attention_fwd(q, k, v, causal=True)
    assert torch.equal(out, st.out)


def test_exact_mode_matches_eq1():
    w = workloads.AttnWorkload("t", 1, 2, 2, 1024, 128, True, 128, 128, seed=9)
    q, k, v = workloads.make_qkv(w)
    st = _run_gpu(w, q.cuda(), k.cuda(), v.cuda(), mode=binding.MODE_EXACT)
    ref = oracle.attention(_np(q), _np(k), _np(v), causal=True, block_q=128, block_k=128, mode=oracle.MODE_EXACT)
    err = np.abs(st.out_f32.cpu().numpy().reshape(ref.out.shape) - ref.out)
    assert err.max() < 2e-2 and err.mean() < 1e-3   # bf16 P in the exact mode


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("D,S", [(128, 128), (128, 640), (64, 1024)])
def test_exp2_setup_small_problems_all_tiles(causal, D, S):
    """The "Exp2 HiF8" setup of Section 4.1 against the checker's version of it."""
    w = workloads.AttnWorkload("t", 2, 4, 2, S, D, causal, 128, 128, seed=40 + S + D + causal)
    _, st, _ = _check(w, what=f"exp2 S={S} D={D} causal={causal}", mode=binding.MODE_EXP2_HIF8)
    assert int(st.restarts.sum()) == 0


def test_exp2_setup_with_outliers_and_rising_max():
    """Outlier keys late in the sequence move the real-valued max in many tiles: exercises the
    rescale of the accumulators by the 8-bit factor."""
    w = workloads.AttnWorkload("t", 1, 4, 2, 2048, 128, False, 128, 128, outlier_frac=0.01, seed=44)
    _check(w, what="exp2 outliers", mode=binding.MODE_EXP2_HIF8)


@pytest.mark.parametrize("name", ["c2_llm_prefill_mha", "c4_vit_encoder"])
def test_exp2_setup_benchmark_configs_full_size_sampled(name):
    w = workloads.WORKLOADS[name]
    _check(w, tiles=workloads.sample_tiles(w)[:8], what="exp2 " + name, mode=binding.MODE_EXP2_HIF8)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("D,S", [(128, 128), (128, 256), (128, 1024), (64, 640)])
def test_b0_first_and_last_small_problems_all_tiles(causal, D, S):
    """B0 = {first, last visible key tile}: tiles visited 0, last, 1, ..., last - 1 (Section 3.2's remark on
    causal language models), one query tile per CTA; every query tile against the checker."""
    w = workloads.AttnWorkload("t", 2, 4, 2, S, D, causal, 128, 128, outlier_frac=0.01, seed=60 + S + D + causal)
    _check(w, what=f"b0 first+last S={S} D={D} causal={causal}", b0_last=True)


def test_b0_first_and_last_full_size_sampled_and_fewer_restarts():
    """On the outlier configuration the second high-precision tile changes the restart counts; the
    sampled tiles must still match the checker, which visits the tiles in the same order."""
    w = workloads.WORKLOADS["c2_llm_prefill_mha"]
    _, st, (qd, kd, vd) = _check(w, tiles=workloads.sample_tiles(w)[:10], what="c2 b0 first+last", b0_last=True)
    base = _run_gpu(w, qd, kd, vd)
    assert not torch.equal(st.restarts, base.restarts)


def test_rising_max_inputs_both_setups_match_the_checker():
    """The accumulated-error experiment's inputs (row maximum rising with every key tile): both
    setups against their checker versions, and the effect itself -- against Eq. (1) the 8-bit
    non-integer rescale factors of the Exp2 setup drift, Algorithm 1's exact factors do not."""
    S, H = 4096, 2
    q, k, v = workloads.make_rising_max_qkv(S, H=H)
    w = workloads.AttnWorkload("rising", 1, H, H, S, 128, False, 128, 128)
    tiles = [(0, 0, 0), (0, 1, 0), (0, 1, S // 128 - 1)]
    qf, kf, vf = _np(q), _np(k), _np(v)
    ex = oracle.attention(qf, kf, vf, causal=False, block_q=128, block_k=128, tiles=np.array(tiles, dtype=np.int32),
                          mode=oracle.MODE_EXACT)
    err = {}
    for mode, omode in ((binding.MODE_E2E_HIF8, oracle.MODE_E2E_HIF8), (binding.MODE_EXP2_HIF8, oracle.MODE_EXP2_HIF8)):
        st = _run_gpu(w, q.cuda(), k.cuda(), v.cuda(), mode=mode)
        ref = oracle.attention(qf, kf, vf, causal=False, block_q=128, block_k=128, mode=omode,
                               tiles=np.array(tiles, dtype=np.int32))
        got = _select(st.out_f32.cpu().numpy(), tiles)
        # every row takes 31 rescale decisions here (the max moves at every tile), each with its own
        # 8-bit rounding boundary: more rows than usual have one of them within 2^-16 of a boundary
        gate_attention(got, ref, what=f"rising max, mode {mode}", max_near_frac=0.10)
        err[mode] = np.abs(got - ex.out).mean()
    assert err[binding.MODE_EXP2_HIF8] > 10 * err[binding.MODE_E2E_HIF8] and err[binding.MODE_E2E_HIF8] < 2e-3


def test_deterministic_run_to_run():
    w = workloads.AttnWorkload("t", 1, 8, 2, 1024, 128, True, 128, 128, seed=10)
    q, k, v = workloads.make_qkv(w, device="cuda")
    a = _run_gpu(w, q, k, v).out_f32.clone()
    for _ in range(3):
        assert torch.equal(_run_gpu(w, q, k, v).out_f32, a)


@pytest.mark.parametrize("name", ["c2_llm_prefill_mha", "c3_llm_prefill_gqa", "c4_vit_encoder"])
def test_benchmark_configs_full_size_sampled(name):
    w = workloads.WORKLOADS[name]
    tiles = workloads.sample_tiles(w)
    _check(w, tiles=tiles, what=name)


def test_long_context_full_size_sampled():
    """The largest configuration, in the launch shape the benchmark times: 26 query tiles -- first,
    second, middle and last of one query head in each of the eight kv groups (other heads of
    the groups for the random ones), the tiles next to the diagonal of a late pair, and six random."""
    w = workloads.WORKLOADS["c5_long_context"]
    nq = w.S // 128
    tiles = set()
    for g in range(w.Hkv):                               # every kv group (4 query heads each)
        h = 4 * g + (g % 4)
        for i in ((0, nq - 1) if g % 2 else (1, nq // 2)):
            tiles.add((0, h, i))
    tiles |= {(0, 0, 0), (0, 31, nq - 1), (0, 30, nq - 2), (0, 9, 100), (0, 17, 200)}
    gen = torch.Generator().manual_seed(7)
    while len(tiles) < 26:
        tiles.add((0, int(torch.randint(0, w.H, (1,), generator=gen)), int(torch.randint(0, nq, (1,), generator=gen))))
    tiles = sorted(tiles)
    assert len({h // 4 for _, h, _ in tiles}) == w.Hkv
    _check(w, tiles=tiles, what="c5 long context")


@pytest.mark.parametrize("lam", [0, 1, 2])
def test_restart_rates_match_checker(lam):
    """ARR / PRR of Table 4 (restarted 8-bit tiles over 8-bit tiles, overall and per query tile)."""
    w = workloads.AttnWorkload("t", 1, 4, 2, 2048, 128, True, 128, 128, outlier_frac=0.01, seed=21 + lam)
    q, k, v = workloads.make_qkv(w)
    out, rates = binding.baps_attention_restart_rates(q.cuda(), k.cuda(), v.cuda(), causal=True, lam=lam)
    binding.poll_async_error()
    ref = oracle.attention(_np(q), _np(k), _np(v), causal=True, block_q=128, block_k=128, lam=lam)
    b1 = (ref.n_tiles - 1).astype(np.float64)
    arr = ref.restarts.sum() / b1.sum()
    prr = np.max(ref.restarts[b1 > 0] / b1[b1 > 0])
    # tiles whose restart decision sat on a rounding boundary may differ
    slack = (ref.row_margin.min(axis=1) < EPS_REL).sum() / b1.sum() + 1e-6
    got = rates.cpu().numpy()
    assert abs(got[0] - arr) <= slack + 1e-6, (got, arr, prr)
    assert abs(got[1] - prr) <= 0.1 * (slack > 1e-5) + 1e-6, (got, arr, prr)
    st = binding.baps_attention_fwd_ex(q.cuda(), k.cuda(), v.cuda(), causal=True, block_q=128, block_k=128, lam=lam)
    assert torch.equal(out, st.out)


def test_restart_rates_rejects_small_scratch():
    w = workloads.AttnWorkload("t", 1, 2, 2, 256, 128, True, 128, 128, seed=3)
    q, k, v = workloads.make_qkv(w, device="cuda")
    with pytest.raises(binding.BapsError):
        binding.baps_attention_restart_rates(q, k, v, causal=True,
                                             scratch=torch.empty(3, dtype=torch.int32, device="cuda"))
