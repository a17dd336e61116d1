"""GPU parity: row softmax (Algorithm 1 on single rows) against the CPU checker."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_02071_b200 import binding, workloads
from parity import gate_softmax_rows

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cols,block_k", [(128, 128), (640, 128), (1024, 128), (1024, 64), (2048, 128), (2048, 64),
                                          (4096, 128), (4096, 64), (8192, 64), (8192, 128), (16384, 64), (32768, 128),
                                          (49152, 128), (65536, 128)])
def test_softmax_rows_matches_checker(cols, block_k):
    rows = 37 if cols <= 8192 else 6
    x = workloads.make_rows(rows, cols, var=4.0, seed=cols + block_k)
    got = binding.baps_softmax_rows(x.cuda(), block_k=block_k).cpu().numpy()
    probs, margin, allow = oracle.softmax_rows(x.numpy(), block_k=block_k, want_allow=True)
    gate_softmax_rows(got, probs, margin, allow, what=f"cols={cols} bk={block_k}")


def test_softmax_rows_increasing_logits_many_restarts():
    """Rows that keep growing force a max update in almost every block."""
    cols = 4096
    base = torch.linspace(-20, 20, cols)[None, :].repeat(8, 1)
    x = base + workloads.make_rows(8, cols, var=1.0, seed=9)
    got = binding.baps_softmax_rows(x.cuda(), block_k=128).cpu().numpy()
    probs, margin, allow = oracle.softmax_rows(x.numpy(), block_k=128, want_allow=True)
    gate_softmax_rows(got, probs, margin, allow, what="increasing")


@pytest.mark.parametrize("cols,block_k,rows", [(1024, 128, 148 * 32 * 16 * 2 + 7), (2048, 128, 148 * 16 * 4 * 3 + 5),
                                               (2048, 64, 148 * 16 * 4 + 1), (4096, 128, 148 * 4 * 4 * 3 + 3),
                                               (8192, 128, 148 * 4 * 4 * 3 + 2), (8192, 64, 148 * 4 * 4 + 3),
                                               (16384, 64, 148 * 2 * 3 + 1), (32768, 128, 148 * 2 * 3 + 2),
                                               (65536, 128, 148 * 2 * 2 + 3), (65536, 64, 148 * 2 + 5)])
def test_softmax_rows_many_rows_per_cta_sampled(cols, block_k, rows):
    """More rows than the grid has row slots (every CTA / group / warp loops, the last pass is ragged),
    with a drift along the row so that some blocks raise the max: sampled rows against the checker, all
    row sums against 1."""
    g = torch.Generator(device="cuda"); g.manual_seed(cols + block_k)
    x = torch.randn(rows, cols, device="cuda", generator=g) * 2.0
    x += torch.linspace(-3, 3, cols, device="cuda")[None, :] * (torch.arange(rows, device="cuda") % 3)[:, None]
    p = binding.baps_softmax_rows(x, block_k=block_k)
    pick = [0, 1, 2, 3, 4, 5, 6, 7, rows // 2, rows // 2 + 1, rows - 6, rows - 5, rows - 4, rows - 3, rows - 2, rows - 1]
    if cols > 16384:
        pick = pick[::2]                         # long rows: the checker takes a second per row
    probs, margin, allow = oracle.softmax_rows(x[pick].cpu().numpy(), block_k=block_k, want_allow=True)
    gate_softmax_rows(p[pick].cpu().numpy(), probs, margin, allow, what=f"many rows cols={cols} bk={block_k}")
    assert float((p.sum(dim=1) - 1).abs().max()) < 1e-4


def test_softmax_rows_full_sweep_size_sampled():
    """2^28 elements as in the benchmark sweep (cols = 16384): check sampled rows one by one."""
    cols = 16384
    rows = (1 << 28) // cols
    g = torch.Generator(device="cuda"); g.manual_seed(11)
    x = torch.randn(rows, cols, device="cuda", generator=g) * 2.0
    p = binding.baps_softmax_rows(x, block_k=128)
    pick = [0, 1, rows // 2, rows - 1, 777]
    probs, margin, allow = oracle.softmax_rows(x[pick].cpu().numpy(), block_k=128, want_allow=True)
    gate_softmax_rows(p[pick].cpu().numpy(), probs, margin, allow, what="sweep sample")
    s = p.sum(dim=1)
    assert float((s - 1).abs().max()) < 1e-4


def _check_codes(x, block_k, what):
    codes, bexp, d = binding.baps_softmax_rows_codes(x.cuda(), block_k=block_k)
    wc, we, wd = oracle.softmax_rows_codes(x.cpu().numpy(), block_k=block_k)
    assert np.array_equal(codes.cpu().numpy(), wc), what            # bit for bit
    assert np.array_equal(bexp.cpu().numpy(), we), what
    assert np.allclose(d.cpu().numpy(), wd, rtol=2e-6, atol=0), what   # fp32 sum against a double sum
    return codes, bexp, d


@pytest.mark.parametrize("cols,block_k", [(128, 128), (640, 128), (1024, 64), (2048, 128), (4096, 64), (8192, 128),
                                          (16384, 128), (49152, 64), (65536, 128)])
def test_softmax_rows_codes_bit_exact(cols, block_k):
    """Row softmax with 8-bit output: HiF8 codes and per-block integer exponents bit for bit."""
    rows = 37 if cols <= 8192 else 5
    x = workloads.make_rows(rows, cols, var=4.0, seed=3 * cols + block_k)
    codes, bexp, d = _check_codes(x, block_k, f"codes cols={cols} bk={block_k}")
    # decoded, the rows sum to one and stay close to the float-output entry point
    p8 = binding.baps_hif8_decode(codes.reshape(-1)).reshape(rows, cols) * \
        torch.exp2(bexp.float()).repeat_interleave(block_k, dim=1) / d[:, None]
    assert float((p8.sum(dim=1) - 1).abs().max()) < 1e-5
    p = binding.baps_softmax_rows(x.cuda(), block_k=block_k)
    # (block 0 is rounded to 8 bits here and kept in fp32 there: up to 2^-4 relative on its weights)
    assert float((p8 - p).abs().max()) < 0.1 * float(p.max())


def test_softmax_rows_codes_increasing_logits_and_full_size_sample():
    cols = 4096
    base = torch.linspace(-20, 20, cols)[None, :].repeat(8, 1)
    _check_codes(base + workloads.make_rows(8, cols, var=1.0, seed=19), 128, "codes increasing")
    # the sweep size: 2^28 elements, sampled rows
    cols = 16384
    rows = (1 << 28) // cols
    g = torch.Generator(device="cuda"); g.manual_seed(12)
    x = torch.randn(rows, cols, device="cuda", generator=g) * 2.0
    codes, bexp, d = binding.baps_softmax_rows_codes(x, block_k=128)
    pick = [0, 1, rows // 2, rows - 1, 4242]
    wc, we, wd = oracle.softmax_rows_codes(x[pick].cpu().numpy(), block_k=128)
    assert np.array_equal(codes[pick].cpu().numpy(), wc) and np.array_equal(bexp[pick].cpu().numpy(), we)
    assert np.allclose(d[pick].cpu().numpy(), wd, rtol=2e-6)


@pytest.mark.parametrize("cols,block_k,rows", [(1024, 128, 148 * 16 * 8 * 2 + 5), (2048, 64, 148 * 16 * 4 * 2 + 3),
                                               (4096, 128, 148 * 4 * 4 * 3 + 1), (8192, 128, 148 * 4 * 4 * 2 + 3),
                                               (16384, 128, 148 * 4 * 2 * 2 + 1), (32768, 64, 148 * 4 * 2 + 1),
                                               (65536, 128, 148 * 2 * 2 + 1)])
def test_softmax_rows_codes_many_rows_per_cta_sampled(cols, block_k, rows):
    """8-bit output with more rows than the grid has row slots: sampled rows bit for bit."""
    g = torch.Generator(device="cuda"); g.manual_seed(7 * cols + block_k)
    x = torch.randn(rows, cols, device="cuda", generator=g) * 2.0
    x += torch.linspace(-3, 3, cols, device="cuda")[None, :] * (torch.arange(rows, device="cuda") % 3)[:, None]
    codes, bexp, d = binding.baps_softmax_rows_codes(x, block_k=block_k)
    pick = [0, 1, 2, 3, 4, 5, 6, 7, rows // 2, rows // 2 + 1, rows - 5, rows - 4, rows - 3, rows - 2, rows - 1]
    wc, we, wd = oracle.softmax_rows_codes(x[pick].cpu().numpy(), block_k=block_k)
    assert np.array_equal(codes[pick].cpu().numpy(), wc)
    assert np.array_equal(bexp[pick].cpu().numpy(), we)
    assert np.allclose(d[pick].cpu().numpy(), wd, rtol=2e-6, atol=0)
    assert bool(torch.isfinite(d).all()) and float(d.min()) > 0


@pytest.mark.parametrize("cols", [1024, 2048, 4096, 8192, 16384, 32768, 65536])
@pytest.mark.parametrize("rows", [1, 3])
def test_softmax_rows_fewer_rows_than_a_cta_holds(cols, rows):
    """One or three rows: groups / warps of the only CTA stay idle; both outputs."""
    x = workloads.make_rows(rows, cols, var=4.0, seed=11 * cols + rows)
    got = binding.baps_softmax_rows(x.cuda(), block_k=128).cpu().numpy()
    probs, margin, allow = oracle.softmax_rows(x.numpy(), block_k=128, want_allow=True)
    gate_softmax_rows(got, probs, margin, allow, what=f"few rows cols={cols} rows={rows}")
    _check_codes(x, 128, f"few rows codes cols={cols} rows={rows}")


@pytest.mark.parametrize("cols", [1024, 2048, 8192, 16384, 32768, 65536])
def test_softmax_rows_staircase_restarts_and_small_rises(cols):
    """Rows whose level jumps by 3 (4.3 in base 2: a restart) at every eighth of the row and creeps up by
    0.4 per sixteenth in between (a rise without restart), so that every kernel variant goes through the
    restart branch, the delta > 0 branch and the positive-T table; both outputs."""
    rows = 5
    pos = torch.arange(cols)
    level = 3.0 * (pos // (cols // 8)).float() + 0.4 * ((pos // (cols // 16)) % 2).float()
    x = level[None, :] + workloads.make_rows(rows, cols, var=0.25, seed=cols + 77)
    for bk in (128, 64):
        got = binding.baps_softmax_rows(x.cuda(), block_k=bk).cpu().numpy()
        probs, margin, allow = oracle.softmax_rows(x.numpy(), block_k=bk, want_allow=True)
        gate_softmax_rows(got, probs, margin, allow, what=f"staircase cols={cols} bk={bk}")
        _check_codes(x, bk, f"staircase codes cols={cols} bk={bk}")


@pytest.mark.parametrize("cols", [1024, 4096, 16384, 65536])
def test_softmax_rows_with_masked_entries(cols):
    """-inf logits (masked positions): scattered ones, and a whole block other than block 0."""
    rows = 4
    x = workloads.make_rows(rows, cols, var=4.0, seed=cols + 5)
    g = torch.Generator(); g.manual_seed(cols)
    x[torch.rand(rows, cols, generator=g) < 0.05] = float("-inf")
    x[:, 256:384] = float("-inf")
    x[:, 0] = 0.5                               # block 0 keeps a finite entry
    got = binding.baps_softmax_rows(x.cuda(), block_k=128).cpu().numpy()
    probs, margin, allow = oracle.softmax_rows(x.numpy(), block_k=128, want_allow=True)
    assert np.isfinite(got).all()
    assert (got[:, 256:384] == 0).all()
    gate_softmax_rows(got, probs, margin, allow, what=f"masked cols={cols}")
    _check_codes(x, 128, f"masked codes cols={cols}")
