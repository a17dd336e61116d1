"""Pins of the CPU checker's Algorithm 1 (attention and row softmax).

Routes that do not go through the checker's own workflow code: Eq. (1) evaluated by numpy,
hand-worked numbers for the max / restart / rescale bookkeeping, invariants (rows sum to one,
V = 1 gives O = 1), special cases that reduce to plain softmax, and brute-force bounds on the
approximation error.
"""
import math

import numpy as np
import pytest

import oracle

LOG2E = 1.4426950408889634


def _exact_attention(q, k, v, causal, scale=None):
    B, H, S, D = q.shape
    Hkv = k.shape[1]
    g = H // Hkv
    scale = 1.0 / math.sqrt(D) if scale is None else scale
    out = np.zeros((B, H, S, D))
    for b in range(B):
        for h in range(H):
            s = (q[b, h].astype(np.float64) @ k[b, h // g].astype(np.float64).T) * scale
            if causal:
                s = np.where(np.tril(np.ones((S, S), bool)), s, -np.inf)
            s -= s.max(axis=1, keepdims=True)
            p = np.exp(s)
            p /= p.sum(axis=1, keepdims=True)
            out[b, h] = p @ v[b, h // g].astype(np.float64)
    return out


def _gather(res, B, H, S, D, bq):
    return res.out.reshape(B, H, S // bq, bq, D).reshape(B, H, S, D)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("bq,bk", [(16, 16), (32, 16), (16, 32), (64, 64), (1, 16)])
@pytest.mark.parametrize("lam", [0, 1, 2])
def test_identity_rounding_reduces_to_eq1(causal, bq, bk, lam):
    """With the 8-bit roundings removed, Algorithm 1 (ceil max, restart branch, the
    power-of-two rescale of the no-restart branch) must be exactly Eq. (1)."""
    rng = np.random.default_rng(10 + lam)
    B, H, Hkv, S, D = 2, 4, 2, 128, 16
    q = (rng.normal(0, 3, (B, H, S, D))).astype(np.float32)
    k = (rng.normal(0, 3, (B, Hkv, S, D))).astype(np.float32)
    v = rng.normal(0, 1, (B, Hkv, S, D)).astype(np.float32)
    res = oracle.attention(q, k, v, causal=causal, block_q=bq, block_k=bk, lam=lam,
                           mode=oracle.MODE_IDENTITY)
    want = _exact_attention(q, k, v, causal)
    assert np.abs(_gather(res, B, H, S, D, bq) - want).max() < 1e-11
    # and the exact mode of the checker is Eq. (1) too
    ex = oracle.attention(q, k, v, causal=causal, block_q=bq, block_k=bk, mode=oracle.MODE_EXACT)
    assert np.abs(_gather(ex, B, H, S, D, bq) - want).max() < 1e-12


def test_single_tile_is_plain_softmax():
    """S <= block_k: only the B0 tile runs, which is Eq. (2) in high precision."""
    rng = np.random.default_rng(3)
    q = rng.normal(0, 2, (1, 2, 64, 32)).astype(np.float32)
    k = rng.normal(0, 2, (1, 2, 64, 32)).astype(np.float32)
    v = rng.normal(0, 1, (1, 2, 64, 32)).astype(np.float32)
    res = oracle.attention(q, k, v, causal=False, block_q=64, block_k=64)
    assert np.abs(_gather(res, 1, 2, 64, 32, 64) - _exact_attention(q, k, v, False)).max() < 1e-12
    assert np.all(res.restarts == 0) and np.all(res.n_tiles == 1)


def test_no_restart_when_max_is_in_first_tile():
    """If every row's largest score lies in key tile 0, T <= 0 in all later tiles: no restart,
    and the final max is ceil of the first tile's row max."""
    rng = np.random.default_rng(4)
    S, D, bk = 256, 32, 32
    q = rng.normal(0, 1, (1, 1, S, D)).astype(np.float32)
    k = rng.normal(0, 1, (1, 1, S, D)).astype(np.float32)
    v = rng.normal(0, 1, (1, 1, S, D)).astype(np.float32)
    s = (q[0, 0].astype(np.float64) @ k[0, 0].astype(np.float64).T) * LOG2E / math.sqrt(D)
    # make key 0 dominate every row: k0 = large multiple of mean query direction won't do for all
    # rows, so build it row-free: scale all other keys down instead.
    k[0, 0, bk:] *= 0.05
    k[0, 0, 0] = 0.0
    s = (q[0, 0].astype(np.float64) @ k[0, 0].astype(np.float64).T) * LOG2E / math.sqrt(D)
    first = s[:, :bk].max(axis=1)
    later = s[:, bk:].max(axis=1)
    keep = first >= later
    assert keep.mean() > 0.9
    res = oracle.attention(q, k, v, causal=False, block_q=1, block_k=bk)
    assert np.all(res.restarts[keep] == 0)
    assert np.array_equal(res.row_m[keep, 0], np.ceil(first[keep]))


def test_value_invariants():
    rng = np.random.default_rng(5)
    B, H, Hkv, S, D = 1, 4, 2, 128, 32
    q = rng.normal(0, 2, (B, H, S, D)).astype(np.float32)
    k = rng.normal(0, 2, (B, Hkv, S, D)).astype(np.float32)
    ones = np.ones((B, Hkv, S, D), np.float32)
    for causal in (False, True):
        res = oracle.attention(q, k, ones, causal=causal, block_q=32, block_k=32)
        assert np.abs(res.out - 1.0).max() < 1e-12


def test_attention_with_identity_values_equals_row_softmax():
    """V = I (D = S) turns O into the probabilities; with block_q = 1 they must equal the
    row-softmax entry point fed with the same scores (ties the two workflows together)."""
    rng = np.random.default_rng(6)
    S = 64
    bk = 16
    # scores chosen directly: q = one-hot rows scaled, k arbitrary => s = c * k[col, row]
    x = rng.normal(0, 2.0, (S, S)).astype(np.float32)            # natural-log logits
    q = np.eye(S, dtype=np.float32)[None, None]
    k = x.T.copy()[None, None]                                    # (q k^T)[r, c] = x[r, c]
    v = np.eye(S, dtype=np.float32)[None, None]
    res = oracle.attention(q, k, v, causal=False, block_q=1, block_k=bk, scale=1.0)
    probs_attn = res.out.reshape(S, S)
    probs_rows = oracle.softmax_rows(x, block_k=bk)
    assert np.abs(probs_attn - probs_rows).max() < 1e-12
    assert np.abs(probs_rows.sum(axis=1) - 1.0).max() < 1e-12


def _row_from_base2(s):
    """natural-log logits (float32) whose base-2 scores are s up to ~1e-7."""
    return (np.asarray(s, dtype=np.float64) / LOG2E).astype(np.float32)[None, :]


def test_hand_worked_no_restart_with_positive_T():
    """Two blocks of one element.  Block 0: s = 0.3 -> m = ceil(0.3) = 1, w0 = 2^-0.7.
    Block 1: s = 1.9 -> T = 0.9 -> HiF8 0.875 (grid 1/16 in [0.5, 1)) <= lambda = 1: no restart;
    delta = ceil(0.875) = 1, m = 2; P8 = HiF8(2^0.875 = 1.834) = 1.875 (grid 1/8 in [1, 2));
    weight relative to the new max = 1.875 / 2; d = w0 / 2 + 0.9375."""
    p = oracle.softmax_rows(_row_from_base2([0.3, 1.9]), block_k=1, lam=1)[0]
    w0 = 2.0 ** -0.7
    d = 0.5 * w0 + 0.9375
    assert np.allclose(p, [0.5 * w0 / d, 0.9375 / d], rtol=0, atol=1e-7)


def test_hand_worked_restart():
    """Block 0: s = 0.3 -> m = 1.  Block 1: s = 3.4 -> T = 2.4 -> HiF8 2.5 (grid 1/4 in [2, 4))
    > lambda = 1: restart; m = max(1, ceil(3.4)) = 4; T = HiF8(-0.6) = -0.625; P8 =
    HiF8(2^-0.625 = 0.6484) = 0.625 (grid 1/16); d = 2^(1-4) * 2^-0.7 + 0.625.
    With lambda = 2 the same input still restarts (2.5 > 2); with lambda = 3 it does not:
    delta = ceil(2.5) = 3, m = 4, P8 = HiF8(2^2.5 = 5.657) = 5.5, weight 5.5 / 8."""
    x = _row_from_base2([0.3, 3.4])
    w0 = 2.0 ** -0.7
    for lam in (1, 2):
        p = oracle.softmax_rows(x, block_k=1, lam=lam)[0]
        d = w0 / 8 + 0.625
        assert np.allclose(p, [w0 / 8 / d, 0.625 / d], rtol=0, atol=1e-7)
    p = oracle.softmax_rows(x, block_k=1, lam=3)[0]
    d = w0 / 8 + 5.5 / 8
    assert np.allclose(p, [w0 / 8 / d, 5.5 / 8 / d], rtol=0, atol=1e-7)


def test_hand_worked_tile_wide_restart_in_attention():
    """The restart test is one decision per tile: a row with T <= lambda takes the restart
    branch because another row of the same query tile exceeds lambda.
    Two query rows, D = 1, scale chosen so that base-2 scores are q * k.
    Row A: s = (0.3, 0.9): alone it would not restart (T = -0.1 -> -0.1015625...).
    Row B: s = (0.3, 3.4): restarts.  In a 2-row tile both rows take the restart branch;
    for row A: m stays max(1, ceil(0.9)) = 1, T = HiF8(0.9 - 1) = HiF8(-0.1) = -0.1015625
    (grid 1/128 in [1/16, 1/8)), P8 = HiF8(2^-0.1015625 = 0.932) = 0.9375."""
    scale = 1.0 / LOG2E
    q = np.array([[[[1.0], [1.0]]]], np.float32)                 # [1,1,2,1]
    k = np.array([[[[0.3], [0.9]]]], np.float32)
    v = np.array([[[[1.0], [0.0]]]], np.float32)
    # separate tiles per row: block_q = 1
    kB = np.array([[[[0.3], [3.4]]]], np.float32)
    # build a 2-row tile whose rows see different scores: use D = 2 with one-hot queries
    q2 = np.array([[[[1.0, 0.0], [0.0, 1.0]]]], np.float32)
    k2 = np.array([[[[0.3, 0.3], [0.9, 3.4]]]], np.float32)
    v2 = np.array([[[[1.0, 0.0], [0.0, 1.0]]]], np.float32)
    res = oracle.attention(q2, k2, v2, causal=False, block_q=2, block_k=1, lam=1, scale=scale)
    assert res.restarts[0] == 1
    w0 = 2.0 ** -0.7
    dA = w0 + 0.9375
    dB = w0 / 8 + 0.625
    want = np.array([[w0 / dA, 0.9375 / dA], [w0 / 8 / dB, 0.625 / dB]])
    assert np.allclose(res.out[0], want, rtol=0, atol=1e-6)
    assert np.array_equal(res.row_m[0], [1.0, 4.0])
    # per-row tiles: row A does not restart and gets the same numbers here (T <= 0, delta = 0)
    resA = oracle.attention(q2, k2, v2, causal=False, block_q=1, block_k=1, lam=1, scale=scale)
    assert list(resA.restarts) == [0, 1]
    assert np.allclose(resA.out.reshape(2, 2), want, rtol=0, atol=1e-6)


def test_causal_mask_hand_case():
    """Row r only sees keys <= r; row 0 of a causal problem returns V[0] exactly."""
    rng = np.random.default_rng(8)
    q = rng.normal(0, 1, (1, 1, 64, 16)).astype(np.float32)
    k = rng.normal(0, 1, (1, 1, 64, 16)).astype(np.float32)
    v = rng.normal(0, 1, (1, 1, 64, 16)).astype(np.float32)
    res = oracle.attention(q, k, v, causal=True, block_q=16, block_k=16)
    out = _gather(res, 1, 1, 64, 16, 16)
    assert np.abs(out[0, 0, 0] - v[0, 0, 0]).max() < 1e-12
    assert list(res.n_tiles) == [1, 2, 3, 4]


def test_softmax_rows_sum_to_one_and_stay_close_to_exact():
    rng = np.random.default_rng(9)
    x = rng.normal(0, 2.0, (64, 1024)).astype(np.float32)
    p = oracle.softmax_rows(x, block_k=128)
    assert np.abs(p.sum(axis=1) - 1).max() < 1e-12
    assert np.all(p >= 0)
    s = x.astype(np.float64) * LOG2E
    ex = np.exp2(s - s.max(axis=1, keepdims=True))
    ex /= ex.sum(axis=1, keepdims=True)
    assert np.abs(p - ex).max() < 4e-2          # the method's own error, not a parity bound
    assert np.abs(p - ex).mean() < 1e-4


def test_weight_error_bound_against_exact_exponential():
    """Brute force on small inputs: every 8-bit-tile weight w (relative to the final integer
    max) against the exact 2^(s - m).  T keeps >= 4 significant bits while |T| < 16, so rounding
    T changes 2^T by at most a factor 2^(|T|/16); T is taken relative to a running max that is
    at most lambda + 1 away from where the score sits relative to the final max; rounding P
    adds a relative half-step of 2^-4 (P >= 2^-3), 2^-3 (P >= 2^-7) or 2^-2 (P >= 2^-15)."""
    rng = np.random.default_rng(13)
    S, bk = 256, 32
    x = rng.normal(0, 2.0, (S, S)).astype(np.float32)
    q = np.eye(S, dtype=np.float32)[None, None]
    k = x.T.copy()[None, None]
    v = np.eye(S, dtype=np.float32)[None, None]
    res = oracle.attention(q, k, v, causal=False, block_q=1, block_k=bk, scale=1.0, lam=1)
    w = res.out.reshape(S, S) * res.row_d.reshape(S, 1)
    t = x.astype(np.float64) * LOG2E - res.row_m.reshape(S, 1)
    w_exact = np.exp2(t)
    sel = (t > -14.0) & (np.arange(S)[None, :] >= bk)
    tt = np.abs(t) + 2.1
    rho = np.where(w_exact >= 2.0 ** -2.9, 2.0 ** -4, np.where(w_exact >= 2.0 ** -6.9, 2.0 ** -3, 0.25))
    hi = np.exp2(tt / 16) * (1 + rho)
    lo = np.exp2(-tt / 16) * (1 - rho)
    ratio = w / w_exact
    assert np.all(ratio[sel] <= hi[sel]) and np.all(ratio[sel] >= lo[sel])
    # B0-tile weights are exact
    assert np.abs(ratio[:, :bk] - 1).max() < 1e-12


def test_attention_error_against_exact_is_small():
    rng = np.random.default_rng(11)
    B, H, Hkv, S, D = 1, 2, 1, 512, 64
    q = rng.normal(0, 1, (B, H, S, D)).astype(np.float32)
    k = rng.normal(0, 1, (B, Hkv, S, D)).astype(np.float32)
    v = rng.normal(0, 1, (B, Hkv, S, D)).astype(np.float32)
    for causal in (False, True):
        res = oracle.attention(q, k, v, causal=causal, block_q=64, block_k=64)
        out = _gather(res, B, H, S, D, 64)
        err = np.abs(out - _exact_attention(q, k, v, causal))
        assert err.max() < 5e-2 and err.mean() < 5e-3
        assert np.all(np.isfinite(res.row_allow)) and np.all(res.row_allow >= 0)


def test_integer_max_and_final_state():
    """The running max is always an integer, never below ceil of the true row max minus the
    slack the restart threshold allows, and d equals the sum of the weights at that max."""
    rng = np.random.default_rng(12)
    S, D = 256, 32
    q = rng.normal(0, 2, (1, 1, S, D)).astype(np.float32)
    k = rng.normal(0, 2, (1, 1, S, D)).astype(np.float32)
    v = rng.normal(0, 1, (1, 1, S, D)).astype(np.float32)
    res = oracle.attention(q, k, v, causal=False, block_q=32, block_k=32, lam=1)
    m = res.row_m.reshape(S)
    assert np.array_equal(m, np.round(m))
    s = (q[0, 0].astype(np.float64) @ k[0, 0].astype(np.float64).T) * LOG2E / math.sqrt(D)
    true_max = s.max(axis=1)
    assert np.all(m >= np.ceil(true_max) - 1)      # T8 <= lambda leaves the max at most ... below
    assert np.all(m <= np.ceil(true_max) + 1)
    assert res.restarts.sum() > 0


def test_argument_validation():
    q = np.zeros((1, 3, 32, 8), np.float32)
    k = np.zeros((1, 2, 32, 8), np.float32)
    with pytest.raises(ValueError):
        oracle.attention(q, k, k, causal=False, block_q=16, block_k=16)
    with pytest.raises(ValueError):
        oracle.softmax_rows(np.zeros((2, 30), np.float32), block_k=16)


# ---- the "Exp2 HiF8" setup of Section 4.1 (Eq. (2) with every 2^x through Algorithm 2) ----------

@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("bq,bk", [(16, 16), (32, 16), (64, 64), (1, 16)])
def test_exp2_setup_with_identity_rounding_reduces_to_eq1(causal, bq, bk):
    """Without the 8-bit conversions the Exp2 setup is plain online softmax, i.e. Eq. (1)."""
    rng = np.random.default_rng(21)
    B, H, Hkv, S, D = 2, 4, 2, 128, 16
    q = rng.normal(0, 3, (B, H, S, D)).astype(np.float32)
    k = rng.normal(0, 3, (B, Hkv, S, D)).astype(np.float32)
    v = rng.normal(0, 1, (B, Hkv, S, D)).astype(np.float32)
    res = oracle.attention(q, k, v, causal=causal, block_q=bq, block_k=bk,
                           mode=oracle.MODE_EXP2_IDENTITY)
    assert np.abs(_gather(res, B, H, S, D, bq) - _exact_attention(q, k, v, causal)).max() < 1e-11


def test_exp2_setup_hand_worked():
    """Three key tiles of one element, base-2 scores (0.3, 1.9, 1.0), real-valued running max.
    Tile 0: m = 0.3, weight EXP2_8(0) = 1, d = 1.
    Tile 1: m = 1.9; rescale factor: HiF8(0.3 - 1.9 = -1.6) = -1.625 (grid 1/8 in [1, 2)),
            2^-1.625 = 0.3242 -> HiF8 0.3125 (grid 1/32 in [1/4, 1/2)); weight EXP2_8(0) = 1;
            d = 0.3125 + 1.
    Tile 2: max unchanged, factor EXP2_8(0) = 1; HiF8(1.0 - 1.9 = -0.9) = -0.875 (grid 1/16 in
            [1/2, 1)), 2^-0.875 = 0.5453 -> HiF8 0.5625 (grid 1/16); d = 1.3125 + 0.5625 = 1.875."""
    scale = 1.0 / LOG2E
    q = np.array([[[[1.0, 0.0, 0.0]] * 3]], np.float32)          # three identical query rows
    k = np.array([[[[0.3, 0, 0], [1.9, 0, 0], [1.0, 0, 0]]]], np.float32)
    v = np.eye(3, dtype=np.float32)[None, None]
    res = oracle.attention(q, k, v, causal=False, block_q=1, block_k=1, scale=scale,
                           mode=oracle.MODE_EXP2_HIF8)
    want = np.array([0.3125, 1.0, 0.5625]) / 1.875
    assert np.allclose(res.out.reshape(3, 3), want[None, :], rtol=0, atol=1e-7)
    assert np.abs(res.row_d - 1.875).max() < 1e-7
    assert np.abs(res.row_m - 1.9).max() < 1e-6


def test_exp2_setup_invariants_and_error():
    rng = np.random.default_rng(22)
    B, H, Hkv, S, D = 1, 4, 2, 256, 32
    q = rng.normal(0, 1.5, (B, H, S, D)).astype(np.float32)
    k = rng.normal(0, 1.5, (B, Hkv, S, D)).astype(np.float32)
    v = rng.normal(0, 1, (B, Hkv, S, D)).astype(np.float32)
    ones = np.ones_like(v)
    for causal in (False, True):
        res = oracle.attention(q, k, ones, causal=causal, block_q=32, block_k=32,
                               mode=oracle.MODE_EXP2_HIF8)
        assert np.abs(res.out - 1.0).max() < 1e-12          # same factors in numerator and d
        res = oracle.attention(q, k, v, causal=causal, block_q=32, block_k=32,
                               mode=oracle.MODE_EXP2_HIF8)
        want = _exact_attention(q, k, v, causal)
        err = np.abs(_gather(res, B, H, S, D, 32) - want)
        # every weight and every rescale factor is within the 8-bit relative error of the exact
        # power, so the output stays close to Eq. (1) -- but it is not equal to it
        assert 1e-4 < err.max() < 0.25 and err.mean() < 0.02
        assert np.all(res.restarts == 0)
    # a single key tile: factor never applied, weights EXP2_8(HiF8(s - m))
    res = oracle.attention(q[:, :, :32], k[:, :, :32], v[:, :, :32], causal=False, block_q=32,
                           block_k=32, mode=oracle.MODE_EXP2_HIF8)
    s = np.einsum("hrd,hcd->hrc", q[0, :, :32].astype(np.float64),
                  np.repeat(k[0, :, :32], 2, axis=0).astype(np.float64)) * LOG2E / math.sqrt(D)
    t = s - s.max(axis=2, keepdims=True)
    w = oracle.hif8_decode(oracle.exp2_code_table()[oracle.hif8_encode(t.astype(np.float64))])
    assert np.abs(res.row_d.reshape(4, 32) - w.sum(axis=2)).max() < 1e-9


def test_integer_rescale_exponents_do_not_accumulate_error():
    """Section 3.3: rescale factors 2^(m_old - m_new) with integer exponents are exact, however many
    times the maximum moves, while factors whose exponent is not an integer and which pass through
    the 8-bit exponential (the Exp2 setup) each carry an 8-bit relative error, and the errors of a
    long chain add up like a random walk.  Built from the checker's primitives alone: rising
    sequences of maxima, the product of the per-step factors against the exact 2^(m_first - m_last)."""
    rng = np.random.default_rng(33)
    tab = oracle.exp2_code_table()
    nseq, nstep = 64, 400
    steps = np.abs(rng.normal(0, 0.7, (nseq, nstep))) + 0.05      # the max rises 400 times
    m_real = np.concatenate([np.zeros((nseq, 1)), np.cumsum(steps, axis=1)], axis=1)
    # integer variant: maxima are ceil'd, the factors are exact powers of two
    m_int = np.ceil(m_real)
    prod_int = np.prod(np.exp2(m_int[:, :-1] - m_int[:, 1:]), axis=1)
    assert np.array_equal(prod_int, np.exp2(m_int[:, 0] - m_int[:, -1]))      # exactly, not approximately
    # non-integer variant: every factor is EXP2_8(HiF8(m_old - m_new))
    expo = m_real[:, :-1] - m_real[:, 1:]
    fac = oracle.hif8_decode(tab[oracle.hif8_encode(expo)])
    one = np.abs(np.log2(fac) - expo)                             # error of a single factor, in the exponent
    assert 0.01 < one.mean() and one.max() < 0.2
    acc = np.abs(np.cumsum(np.log2(fac) - expo, axis=1))          # accumulated error after n updates
    assert acc[:, -1].mean() > 2.5 * acc[:, 24].mean()            # ~ sqrt(400 / 25) = 4 for a random walk
    assert acc[:, -1].mean() > 0.3                                # i.e. > 20 % relative error on average


# ---- pins of the two arrays that widen the GPU parity gate: row_allow and row_margin --------------
# Both are computed inside the checker; the expected values below are worked out by hand from the
# float32 inputs actually passed in (so that the input rounding is accounted for), never from the
# checker's own code.

def _one_row_attention(scores, values, lam=1):
    """One query row, one key per tile, D = 1: base-2 scores are the float32 k values themselves."""
    n = len(scores)
    q = np.ones((1, 1, n, 1), np.float32)            # every row identical; row n-1 sees all keys
    k = np.asarray(scores, np.float32).reshape(1, 1, n, 1)
    v = np.asarray(values, np.float32).reshape(1, 1, n, 1)
    res = oracle.attention(q, k, v, causal=False, block_q=1, block_k=1, lam=lam, scale=1.0 / LOG2E,
                           tiles=np.array([[0, 0, n - 1]], np.int32))
    return res, k.reshape(n).astype(np.float64), v.reshape(n).astype(np.float64)


def test_row_allow_hand_worked_single_near_boundary_element():
    """Tile 1's T = s1 - 1 sits a relative 2^-20 inside the HiF8 rounding midpoint 0.59375 (between
    0.5625 and 0.625, grid 1/16): it rounds to -0.5625, weight HiF8(2^-0.5625 = 0.677) = 0.6875; on
    the other side it would be -0.625, weight HiF8(0.648) = 0.625: |dw| = 0.0625.  No other element
    is near a boundary, the max never moves (m = 1), so
        row_allow = |dw| * |v1 - out| / (d - |dw|)."""
    s1 = 1.0 - 0.59375 * (1.0 - 2.0 ** -20)
    res, s, v = _one_row_attention([0.3, s1, -1.0], [0.25, -1.5, 2.0])
    t1 = s[1] - 1.0
    assert -0.59375 < t1 and abs(t1 + 0.59375) < 2.0 ** -16          # really on the 0.5625 side, really near
    w = np.array([2.0 ** (s[0] - 1.0), 0.6875, 0.25])                # B0 weight exact; HiF8(2^-2) = 0.25
    d = w.sum()
    out = (w * v).sum() / d
    assert abs(res.out[0, 0, 0] - out) < 1e-12 and abs(res.row_d[0, 0] - d) < 1e-12
    want = 0.0625 * abs(v[1] - out) / (d - 0.0625)
    assert abs(res.row_allow[0, 0] - want) < 1e-12 and want > 0.03
    # moved away from the midpoint: nothing is near, the allowance is exactly zero
    res2, _, _ = _one_row_attention([0.3, 1.0 - 0.58, -1.0], [0.25, -1.5, 2.0])
    assert res2.row_allow[0, 0] == 0.0
    # just outside the window (relative 2^-15 from the midpoint): zero as well
    res3, s3, _ = _one_row_attention([0.3, 1.0 - 0.59375 * (1.0 - 2.0 ** -15), -1.0], [0.25, -1.5, 2.0])
    assert abs(s3[1] - 1.0 + 0.59375) > 2.0 ** -16 and res3.row_allow[0, 0] == 0.0


def test_row_allow_scales_with_later_rescale_and_row_margin_value():
    """Same near-boundary element, then a tile that restarts and lifts the max from 1 to 3: the
    ambiguous weight change is carried at 2^(1-3), and d is the final denominator.
    Tile 3: s = 2.5, T = 1.5 > lambda: restart, m = 3, T = HiF8(-0.5) = -0.5, weight HiF8(0.7071) =
    0.6875.  Decision margins of the row: tile 0 max 0.3 is 0.3 from the integer 0; the restart max
    2.5 is 0.5 from 2 and 3, relative to |2.5|: 0.2 -- the smallest, so row_margin = 0.2."""
    s1 = 1.0 - 0.59375 * (1.0 - 2.0 ** -20)
    res, s, v = _one_row_attention([0.3, s1, -1.0, 2.5], [0.25, -1.5, 2.0, 0.5])
    w = np.array([2.0 ** (s[0] - 1.0), 0.6875, 0.25]) / 4.0
    w = np.append(w, 0.6875)
    d = w.sum()
    out = (w * v).sum() / d
    assert abs(res.out[0, 0, 0] - out) < 1e-12 and res.restarts[0] == 1 and res.row_m[0, 0] == 3.0
    want = (0.0625 / 4) * abs(v[1] - out) / (d - 0.0625 / 4)
    assert abs(res.row_allow[0, 0] - want) < 1e-12
    assert abs(res.row_margin[0, 0] - 0.2) < 1e-9


def test_row_margin_zero_when_row_max_sits_on_an_integer():
    """B0 tile: m = ceil(rowmax S); a row max exactly on an integer has margin 0, one that is a
    distance e below it has margin e / |max|."""
    res, _, _ = _one_row_attention([2.0, 0.5], [1.0, 0.0])
    assert res.row_margin[0, 0] == 0.0
    res, s, _ = _one_row_attention([2.0 - 2.0 ** -20, 0.5], [1.0, 0.0])
    assert abs(res.row_margin[0, 0] - (2.0 - s[0]) / s[0]) < 1e-15 and res.row_margin[0, 0] > 0


def test_row_margin_when_tile_max_sits_on_the_lambda_midpoint():
    """lambda = 1: the restart test flips where HiF8(T) leaves 1.0 for 1.125, i.e. at T = 1.0625.
    T a relative 2^-20 below it: no restart, delta = ceil(1.0) = 1; on the other side the tile would
    restart and delta would be 2 -- both decisions have the same margin, |T - 1.0625| / |s|."""
    s1 = 1.0 + 1.0625 * (1.0 - 2.0 ** -20)
    res, s, _ = _one_row_attention([0.3, s1], [1.0, 0.0])
    t = s[1] - 1.0
    assert t < 1.0625 and res.restarts[0] == 0 and res.row_m[0, 0] == 2.0
    assert abs(res.row_margin[0, 0] - (1.0625 - t) / s[1]) < 1e-12
    assert res.row_margin[0, 0] < 2.0 ** -16
    # a hair above the midpoint: restart, and the margin is the same distance from the other side
    res, s, _ = _one_row_attention([0.3, 1.0 + 1.0625 * (1.0 + 2.0 ** -20)], [1.0, 0.0])
    t = s[1] - 1.0
    assert t > 1.0625 and res.restarts[0] == 1 and res.row_m[0, 0] == 3.0
    assert abs(res.row_margin[0, 0] - (t - 1.0625) / s[1]) < 1e-12


def test_softmax_rows_allow_and_margin_hand_worked():
    """Row softmax, blocks of one element, same construction: block 1 has T within 2^-20 (relative)
    of the midpoint 0.59375.  With a = |dw| / d (the normalised ambiguous weight change, 0.0625 / d),
        allow[c] = (own change + p[c] * a) / (1 - a):  own change = a for c = 1, 0 elsewhere.
    Decision margin of the row: block 0's max 0.3 (0.3 from an integer); the other blocks have
    T < 0 on both sides of their boundary, which changes neither the restart test nor delta."""
    s1 = 1.0 - 0.59375 * (1.0 - 2.0 ** -20)
    x = _row_from_base2([0.3, s1, -1.0])
    s = x[0].astype(np.float64) * LOG2E
    assert abs((s[1] - 1.0) + 0.59375) < 2.0 ** -16 and s[1] - 1.0 > -0.59375
    p, margin, allow = oracle.softmax_rows(x, block_k=1, lam=1, want_allow=True)
    w = np.array([2.0 ** (s[0] - 1.0), 0.6875, 0.25])
    d = w.sum()
    assert np.abs(p[0] - w / d).max() < 1e-12
    a = 0.0625 / d
    want = (np.array([0.0, a, 0.0]) + (w / d) * a) / (1.0 - a)
    assert np.abs(allow[0] - want).max() < 1e-12
    assert abs(margin[0] - 0.3) < 1e-6
    # nothing near a boundary: allowance exactly zero
    p, margin, allow = oracle.softmax_rows(_row_from_base2([0.3, 0.42, -1.0]), block_k=1, lam=1, want_allow=True)
    assert np.all(allow == 0.0)
    # block maximum on the lambda midpoint: margin = |T - 1.0625| / |s|
    x = _row_from_base2([0.3, 1.0 + 1.0625 * (1.0 - 2.0 ** -20)])
    s = x[0].astype(np.float64) * LOG2E
    _, margin, _ = oracle.softmax_rows(x, block_k=1, lam=1, want_allow=True)
    assert abs(margin[0] - (1.0625 - (s[1] - 1.0)) / s[1]) < 1e-12 and margin[0] < 2.0 ** -16
    # block 0's maximum exactly on an integer: margin 0
    _, margin, _ = oracle.softmax_rows(np.array([[2.0 / LOG2E, 0.1]], np.float64).astype(np.float32), block_k=1,
                                       lam=1, want_allow=True)
    assert margin[0] < 1e-6


# ---- B0 = {first, last visible key tile} (Section 3.2's remark on causal language models) -----------

@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("bq,bk", [(16, 16), (32, 16), (64, 64), (1, 16)])
def test_b0_first_and_last_with_identity_rounding_reduces_to_eq1(causal, bq, bk):
    """The visiting order 0, last, 1, ..., last - 1 with two high-precision tiles is still Eq. (1)
    once the 8-bit roundings are removed."""
    rng = np.random.default_rng(41)
    B, H, Hkv, S, D = 2, 4, 2, 128, 16
    q = rng.normal(0, 3, (B, H, S, D)).astype(np.float32)
    k = rng.normal(0, 3, (B, Hkv, S, D)).astype(np.float32)
    v = rng.normal(0, 1, (B, Hkv, S, D)).astype(np.float32)
    res = oracle.attention(q, k, v, causal=causal, block_q=bq, block_k=bk, mode=oracle.MODE_IDENTITY, b0_last=True)
    assert np.abs(_gather(res, B, H, S, D, bq) - _exact_attention(q, k, v, causal)).max() < 1e-11


def test_b0_first_and_last_hand_worked():
    """One row, three tiles of one key, base-2 scores (0.3, 1.9, 3.4).  Order 0, 2, 1:
    tile 0: m = ceil(0.3) = 1, w = 2^-0.7;   tile 2 (B0 as well): m = max(1, ceil(3.4)) = 4, the old sum
    is scaled by 2^-3, w = 2^(3.4 - 4) in high precision;   tile 1 (8-bit): T = 1.9 - 4 = -2.1 -> HiF8 -2
    (grid 1/4 in [2, 4)), P8 = HiF8(2^-2) = 0.25, no restart, delta = 0.
    With B0 = {first} the same input restarts at the last tile instead (test_hand_worked_restart style):
    the two results differ."""
    res, s, v = None, None, None
    q = np.ones((1, 1, 3, 1), np.float32)
    k = np.array([0.3, 1.9, 3.4], np.float32).reshape(1, 1, 3, 1)
    vv = np.array([1.0, -2.0, 0.5], np.float32).reshape(1, 1, 3, 1)
    kw = dict(causal=False, block_q=1, block_k=1, scale=1.0 / LOG2E, tiles=np.array([[0, 0, 2]], np.int32))
    res = oracle.attention(q, k, vv, b0_last=True, **kw)
    s = k.reshape(3).astype(np.float64)
    w = np.array([2.0 ** (s[0] - 1.0) / 8.0, 0.25, 2.0 ** (s[2] - 4.0)])
    d = w.sum()
    assert abs(res.row_d[0, 0] - d) < 1e-12 and res.row_m[0, 0] == 4.0
    assert abs(res.out[0, 0, 0] - (w * vv.reshape(3)).sum() / d) < 1e-12
    assert res.restarts[0] == 0 and res.n_tiles[0] == 3
    first_only = oracle.attention(q, k, vv, b0_last=False, **kw)
    assert first_only.restarts[0] == 1 and abs(first_only.out[0, 0, 0] - res.out[0, 0, 0]) > 1e-3


def test_b0_first_and_last_edge_cases():
    """Two visible tiles: both are B0, the result is plain softmax; one tile: nothing changes.  Causal:
    "last" is the diagonal tile of each query tile, and the large scores there no longer restart."""
    rng = np.random.default_rng(42)
    q = rng.normal(0, 2, (1, 2, 64, 16)).astype(np.float32)
    k = rng.normal(0, 2, (1, 2, 64, 16)).astype(np.float32)
    v = rng.normal(0, 1, (1, 2, 64, 16)).astype(np.float32)
    two = oracle.attention(q, k, v, causal=False, block_q=32, block_k=32, b0_last=True)
    assert np.abs(_gather(two, 1, 2, 64, 16, 32) - _exact_attention(q, k, v, False)).max() < 1e-12
    one = oracle.attention(q[:, :, :32], k[:, :, :32], v[:, :, :32], causal=False, block_q=32, block_k=32, b0_last=True)
    ref = oracle.attention(q[:, :, :32], k[:, :, :32], v[:, :, :32], causal=False, block_q=32, block_k=32)
    assert np.array_equal(one.out, ref.out)
    # causal with a recency bias: keys close to the query score high (diagonal tile), as in language models
    S, D, b = 256, 16, 16
    q = rng.normal(0, 1, (1, 1, S, D)).astype(np.float32)
    k = rng.normal(0, 1, (1, 1, S, D)).astype(np.float32)
    v = rng.normal(0, 1, (1, 1, S, D)).astype(np.float32)
    q[..., 0] = 6.0
    k[..., 0] = np.linspace(0.0, 6.0, S)[None, None, :]          # score grows with the key position
    a = oracle.attention(q, k, v, causal=True, block_q=b, block_k=b)
    c = oracle.attention(q, k, v, causal=True, block_q=b, block_k=b, b0_last=True)
    assert a.restarts.sum() > 0 and c.restarts.sum() < a.restarts.sum()
    want = _exact_attention(q, k, v, True)
    assert np.abs(_gather(c, 1, 1, S, D, b) - want).max() < 0.1
