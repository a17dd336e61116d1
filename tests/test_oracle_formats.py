"""Pins of the comparison setups of Section 4.2 in the CPU checker: the Exp2 setup with E4M3 /
E5M2 / E4M3-in-E5M2-out exponentials, and "Naive E2E".  The FP8 roundings are checked against
torch's float8 casts (an independent encoder), the setups against hand-worked numbers and against
the same formulas evaluated with torch casts."""
import math

import numpy as np
import pytest
import torch

import oracle

LOG2E = 1.4426950408889634


def _torch_e4m3(x):
    return torch.tensor(np.asarray(x, np.float64), dtype=torch.float32).to(torch.float8_e4m3fn).to(torch.float64).numpy()


def _torch_e5m2(x):
    return torch.tensor(np.asarray(x, np.float64), dtype=torch.float32).to(torch.float8_e5m2).to(torch.float64).numpy()


def test_fp8_roundings_match_torch_casts():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(0, 1, 4000), rng.normal(0, 50, 2000), np.exp2(rng.uniform(-18, 8, 4000)),
                        -np.exp2(rng.uniform(-18, 8, 2000)), [0.0, 2.0 ** -9, 2.0 ** -10, 1.5 * 2.0 ** -9, 2.0 ** -16,
                                                             2.0 ** -17, 1.0625, 1.1875, 440.0, 3.0 * 2.0 ** -17]])
    x = x.astype(np.float32).astype(np.float64)                      # values a float32 cast can be fed with
    inside4 = np.abs(x) <= 448.0                                     # beyond: the checker saturates, torch gives NaN
    assert np.array_equal(oracle.round_e4m3(x[inside4]), _torch_e4m3(x[inside4]))
    inside5 = np.abs(x) <= 57344.0
    assert np.array_equal(oracle.round_e5m2(x[inside5]), _torch_e5m2(x[inside5]))
    # saturation (reading: finite input never becomes NaN or infinity)
    assert oracle.round_e4m3([1e4, -1e4]).tolist() == [448.0, -448.0]
    assert oracle.round_e5m2([1e9, -1e9]).tolist() == [57344.0, -57344.0]


def test_e4m3_has_no_resolution_below_two_to_minus_nine():
    """Section 3.1: for P in [0, 2^-9) E4M3 has nothing to offer (its smallest value is 2^-9), E5M2
    goes down to 2^-16 -- the reason E5M2 suits the result of the exponential and E4M3 its argument."""
    assert oracle.round_e4m3([2.0 ** -10, 2.0 ** -11, 0.9 * 2.0 ** -9]).tolist() == [0.0, 0.0, 2.0 ** -9]
    assert oracle.round_e5m2([2.0 ** -10, 2.0 ** -11, 2.0 ** -16]).tolist() == [2.0 ** -10, 2.0 ** -11, 2.0 ** -16]
    # and E4M3 resolves the argument better: T = -0.3 -> -0.3125 (3 mantissa bits) vs -0.3125 / -0.25 grid of E5M2
    assert oracle.round_e4m3([-0.3])[0] == -0.3125 and oracle.round_e5m2([-0.3])[0] == -0.3125
    assert oracle.round_e4m3([-0.34])[0] == -0.34375 and oracle.round_e5m2([-0.34])[0] == -0.3125


def _two_key_problem(s0, s1):
    q = np.ones((1, 1, 2, 1), np.float32)
    k = np.array([s0, s1], np.float32).reshape(1, 1, 2, 1)
    v = np.array([1.0, 0.0], np.float32).reshape(1, 1, 2, 1)
    return q, k, v, dict(causal=False, block_q=1, block_k=1, scale=1.0 / LOG2E, tiles=np.array([[0, 0, 1]], np.int32))


def test_naive_e2e_hand_worked():
    """Scores (5.3, 5.0) are sent as HiF8 first: 5.5 and 5.0 (grid 1/2 in [4, 8)).  Tile 0: m = 5.5, weight
    EXP2_8(0) = 1.  Tile 1: max unchanged; T = 5.0 - 5.5 = -0.5, 2^-0.5 = 0.7071 -> HiF8 0.6875: d = 1.6875.
    The Exp2 HiF8 setup on the same input subtracts first: T = HiF8(5.0 - 5.3) = -0.3125 (grid 1/32),
    2^-0.3125 = 0.805 -> 0.8125: d = 1.8125 (exact: 1 + 2^-0.3 = 1.812)."""
    q, k, v, kw = _two_key_problem(5.3, 5.0)
    naive = oracle.attention(q, k, v, mode=oracle.MODE_NAIVE_E2E, **kw)
    assert abs(naive.row_d[0, 0] - 1.6875) < 1e-12 and abs(naive.out[0, 0, 0] - 1 / 1.6875) < 1e-12
    exp2 = oracle.attention(q, k, v, mode=oracle.MODE_EXP2_HIF8, **kw)
    assert abs(exp2.row_d[0, 0] - 1.8125) < 1e-12


def test_fp8_exp2_setups_hand_worked():
    """Scores (2.0, -8.3), real-valued max 2.0 after tile 0 (weight 2^0 = 1 in every format).
    Tile 1: T = -10.3.  E4M3: -10 (grid 1 in [8, 16)), 2^-10 -> E4M3 0 (nothing below 2^-9): d = 1.
    E5M2: -10 (grid 2: -10.3 -> -10), 2^-10 exactly: d = 1 + 2^-10.  E4M3 in, E5M2 out: the same."""
    q, k, v, kw = _two_key_problem(2.0, -8.3)
    for mode, want in ((oracle.MODE_EXP2_E4M3, 1.0), (oracle.MODE_EXP2_E5M2, 1.0 + 2.0 ** -10),
                       (oracle.MODE_EXP2_E4M3_E5M2, 1.0 + 2.0 ** -10)):
        res = oracle.attention(q, k, v, mode=mode, **kw)
        assert abs(res.row_d[0, 0] - want) < 1e-15, mode


@pytest.mark.parametrize("mode,fin,fout", [(5, _torch_e4m3, _torch_e4m3), (6, _torch_e5m2, _torch_e5m2),
                                           (7, _torch_e4m3, _torch_e5m2)])
def test_fp8_exp2_setups_single_tile_against_torch_casts(mode, fin, fout):
    """One key tile: no rescale factor is ever applied, the weights are out(2^in(s - rowmax)) and the
    denominator is their sum -- evaluated here with torch's casts."""
    rng = np.random.default_rng(mode)
    S, D = 32, 16
    q = rng.normal(0, 2, (1, 2, S, D)).astype(np.float32)
    k = rng.normal(0, 2, (1, 2, S, D)).astype(np.float32)
    v = rng.normal(0, 1, (1, 2, S, D)).astype(np.float32)
    res = oracle.attention(q, k, v, causal=False, block_q=S, block_k=S, mode=mode)
    s = np.einsum("hrd,hcd->hrc", q[0].astype(np.float64), k[0].astype(np.float64)) * LOG2E / math.sqrt(D)
    t = (s - s.max(axis=2, keepdims=True)).astype(np.float32).astype(np.float64)
    # (float32 so that torch can be fed; skip rows where that cast moved a value across a rounding boundary)
    w = fout(np.exp2(fin(t)).astype(np.float32))
    d = w.sum(axis=2)
    ok = np.abs(res.row_d.reshape(2, S) - d) < 1e-9
    assert ok.mean() > 0.9
    ones = np.ones_like(v)
    res1 = oracle.attention(q, k, ones, causal=False, block_q=S, block_k=S, mode=mode)
    assert np.abs(res1.out - 1.0).max() < 1e-12


def test_setups_error_ordering_on_synthetic_scores():
    """Error against Eq. (1) on unit-Gaussian inputs with a few outlier keys (large scores): casting the
    scores before the subtraction (Naive E2E) costs far more than Algorithm 1, because HiF8 keeps only
    one or two mantissa bits where the raw scores are large; E4M3 in and out loses the small weights."""
    rng = np.random.default_rng(5)
    B, H, S, D = 1, 2, 1024, 64
    q = rng.normal(0, 1, (B, H, S, D)).astype(np.float32)
    k = rng.normal(0, 1, (B, H, S, D)).astype(np.float32)
    v = rng.normal(0, 1, (B, H, S, D)).astype(np.float32)
    k[:, :, rng.choice(S, 10, replace=False)] *= 8.0
    tiles = np.array([[0, 0, 3], [0, 1, 7]], np.int32)
    kw = dict(causal=True, block_q=128, block_k=128, tiles=tiles)
    ex = oracle.attention(q, k, v, mode=oracle.MODE_EXACT, **kw).out
    err = {}
    for name, mode in (("e2e", oracle.MODE_E2E_HIF8), ("exp2", oracle.MODE_EXP2_HIF8), ("e4m3", oracle.MODE_EXP2_E4M3),
                       ("e5m2", oracle.MODE_EXP2_E5M2), ("e4m3xe5m2", oracle.MODE_EXP2_E4M3_E5M2),
                       ("naive", oracle.MODE_NAIVE_E2E)):
        err[name] = np.abs(oracle.attention(q, k, v, mode=mode, **kw).out - ex).mean()
    assert err["naive"] > 3 * err["e2e"], err
    assert err["naive"] > 3 * err["exp2"], err
    assert err["e4m3xe5m2"] < err["e5m2"], err            # finer arguments help
    for name in err:
        assert np.isfinite(err[name]) and err[name] < 0.5, err


# ---- row softmax with 8-bit output (HiF8 codes + per-block integer exponents) ----------------------

def test_softmax_rows_codes_hand_worked():
    """Blocks of one element, base-2 scores (0.3, 1.9, 3.4, -1.0), lambda = 1 (cf. the hand-worked cases of
    the float-output version).  Block 0: m = 1, T = HiF8(-0.7) = -0.6875, code of HiF8(2^-0.6875 = 0.621) = 0.625.
    Block 1: T = 0.9 -> 0.875 <= 1: no restart, code of HiF8(2^0.875 = 1.834) = 1.875, T against m = 1, then
    m = 2.  Block 2: T = 1.4 -> 1.375 > 1: restart, m = 4, T = HiF8(-0.6) = -0.625, code of 0.625.
    Block 3: T = -5 -> code of HiF8(2^-5) = 2^-5.  Exponents mref - m_final: (1, 1, 4, 4) - 4."""
    x = (np.array([[0.3, 1.9, 3.4, -1.0]]) / LOG2E).astype(np.float32)
    codes, bexp, d = oracle.softmax_rows_codes(x, block_k=1, lam=1)
    vals = oracle.hif8_decode(codes[0])
    assert vals.tolist() == [0.625, 1.875, 0.625, 2.0 ** -5]
    assert bexp[0].tolist() == [-3, -3, 0, 0]
    assert abs(d[0] - (0.625 / 8 + 1.875 / 8 + 0.625 + 2.0 ** -5)) < 1e-12


def test_softmax_rows_codes_consistent_with_float_version():
    """Decoded, the 8-bit output is the float-output row softmax up to what differs by construction: block 0
    goes through the 8-bit exponential (one HiF8 rounding of its weights, <= 2^-4 relative) and T is formed in
    single precision.  Rows sum to one exactly in the decoded form."""
    rng = np.random.default_rng(17)
    x = rng.normal(0, 2.0, (64, 2048)).astype(np.float32)
    codes, bexp, d = oracle.softmax_rows_codes(x, block_k=128)
    p8 = oracle.hif8_decode(codes) * np.exp2(np.repeat(bexp, 128, axis=1).astype(np.float64)) / d[:, None]
    assert np.abs(p8.sum(axis=1) - 1.0).max() < 1e-12
    p = oracle.softmax_rows(x, block_k=128)
    assert np.abs(p8 - p).max() < 2e-2 and np.abs(p8 - p).mean() < 1e-4
    assert np.all(bexp <= 0)
    # beyond block 0 the two versions form the same weights; only the denominators differ (block 0), so
    # the ratio of the probabilities is one constant per row wherever single and double precision T round alike
    ratio = p8[:, 128:] / np.where(p[:, 128:] > 0, p[:, 128:], 1.0)
    med = np.median(ratio, axis=1, keepdims=True)
    assert (np.abs(ratio / med - 1.0) < 1e-9).mean() > 0.99
