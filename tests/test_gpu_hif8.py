"""GPU parity: HiF8 encode / decode / 8-bit exponent against the CPU checker, bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_02071_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def _structured_inputs():
    table = oracle.hif8_value_table()
    fin = np.sort(table[np.isfinite(table)])
    pts = [fin]
    mids = 0.5 * (fin[:-1] + fin[1:])
    f32 = lambda a: np.asarray(a, dtype=np.float32)
    pts += [f32(mids), np.nextafter(f32(mids), np.float32(np.inf)), np.nextafter(f32(mids), np.float32(-np.inf))]
    pts += [np.nextafter(f32(fin), np.float32(np.inf)), np.nextafter(f32(fin), np.float32(-np.inf))]
    pts += [f32([40960.0, 40959.9, -40960.0, 65504.0, 1e30, -1e30, np.inf, -np.inf, np.nan,
                 2.0 ** -23, -(2.0 ** -23), 0.999 * 2.0 ** -23, 2.0 ** -24, 1e-45, -1e-45, 0.0, -0.0])]
    pts += [f32(np.exp2(np.arange(-30, 20, dtype=np.float64)))]
    return np.concatenate([f32(p) for p in pts])


def test_encode_structured_and_random_bit_exact():
    rng = np.random.default_rng(0)
    x = np.concatenate([
        _structured_inputs(),
        rng.normal(0, 2, 1 << 20).astype(np.float32),
        (np.exp2(rng.uniform(-26, 17, 1 << 20)) * rng.choice([-1, 1], 1 << 20)).astype(np.float32),
    ])
    x = x[: len(x) - 5]                      # ragged length (not a multiple of 16)
    xd = torch.from_numpy(x).cuda()
    got = binding.baps_hif8_encode(xd).cpu().numpy()
    want = oracle.hif8_encode(x.astype(np.float64))
    assert np.array_equal(got, want)


def test_encode_every_fp32_prefix_bit_exact():
    """Every (sign, exponent, top-7-mantissa) prefix, with the low bits all zero and all one."""
    hi = (np.arange(1 << 16, dtype=np.uint32) << 16)
    bits = np.concatenate([hi, hi | np.uint32(0xFFFF)])
    x = bits.view(np.float32)
    got = binding.baps_hif8_encode(torch.from_numpy(x).cuda()).cpu().numpy()
    want = oracle.hif8_encode(x.astype(np.float64))
    assert np.array_equal(got, want)


def test_decode_all_codes_and_round_trip():
    codes = np.tile(np.arange(256, dtype=np.uint8), 41)[:-3]
    got = binding.baps_hif8_decode(torch.from_numpy(codes).cuda()).cpu().numpy()
    want = oracle.hif8_decode(codes)
    assert np.array_equal(np.isnan(got), np.isnan(want))
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok].astype(np.float64), want[ok])
    back = binding.baps_hif8_encode(torch.from_numpy(got).cuda()).cpu().numpy()
    assert np.array_equal(back, codes)


def test_exp2_all_codes_bit_exact():
    codes = np.tile(np.arange(256, dtype=np.uint8), 33)[:-7]
    got = binding.baps_exp2_hif8(torch.from_numpy(codes).cuda()).cpu().numpy()
    want = oracle.exp2_code_table()[codes]
    assert np.array_equal(got, want)


def test_empty_and_tiny_inputs():
    e = torch.empty(0, dtype=torch.float32, device="cuda")
    assert binding.baps_hif8_encode(e).numel() == 0
    x = torch.tensor([1.0625, -5.3, 100.0], device="cuda")
    assert binding.baps_hif8_encode(x).cpu().tolist() == [0x09, 0xA3, 0x4A]


def test_encode_large_buffer_sampled():
    """Full sweep size (2^28 elements, the size the benchmark times): check a strided sample."""
    n = 1 << 28
    g = torch.Generator(device="cuda"); g.manual_seed(5)
    x = torch.randn(n, device="cuda", generator=g) * 2.0
    codes = binding.baps_hif8_encode(x)
    idx = torch.arange(0, n, 4099, device="cuda")
    xs = x[idx].cpu().numpy(); cs = codes[idx].cpu().numpy()
    assert np.array_equal(cs, oracle.hif8_encode(xs.astype(np.float64)))
    tail = slice(n - 1000, n)
    assert np.array_equal(codes[tail].cpu().numpy(), oracle.hif8_encode(x[tail].cpu().numpy().astype(np.float64)))


@pytest.mark.parametrize("n", [16384 * 5 + 16 * 37 + 9, 16384 * 2, 16384 + 15, 1 << 22])
def test_decode_whole_iterations_and_ragged_tail(n):
    """Several whole CTA iterations (16384 codes each) plus a ragged rest, random codes."""
    rng = np.random.default_rng(n)
    codes = rng.integers(0, 256, n, dtype=np.uint8)
    got = binding.baps_hif8_decode(torch.from_numpy(codes).cuda()).cpu().numpy()
    want = oracle.hif8_decode(codes)
    assert np.array_equal(np.isnan(got), np.isnan(want))
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok].astype(np.float64), want[ok])


@pytest.mark.parametrize("n", [32768 * 3 + 16 * 100 + 7, 32768 * 2, 32768 + 16, (1 << 22) + 5])
def test_exp2_whole_iterations_and_ragged_tail(n):
    rng = np.random.default_rng(n)
    codes = rng.integers(0, 256, n, dtype=np.uint8)
    got = binding.baps_exp2_hif8(torch.from_numpy(codes).cuda()).cpu().numpy()
    assert np.array_equal(got, oracle.exp2_code_table()[codes])


@pytest.mark.parametrize("n", [16384 * 3 + 4 * 77 + 3, 16384 * 2, 16384 + 1])
def test_encode_whole_iterations_and_ragged_tail(n):
    rng = np.random.default_rng(n)
    x = rng.normal(0, 2, n).astype(np.float32)
    got = binding.baps_hif8_encode(torch.from_numpy(x).cuda()).cpu().numpy()
    assert np.array_equal(got, oracle.hif8_encode(x.astype(np.float64)))


def test_decode_and_exp2_large_buffer_sampled():
    """Sweep size (2^28 codes, as the benchmark times them): a strided sample and both ends."""
    n = 1 << 28
    g = torch.Generator(device="cuda"); g.manual_seed(6)
    codes = torch.randint(0, 256, (n,), dtype=torch.uint8, device="cuda", generator=g)
    vals = binding.baps_hif8_decode(codes)
    p = binding.baps_exp2_hif8(codes)
    idx = torch.cat([torch.arange(0, n, 4099, device="cuda"), torch.arange(0, 70000, device="cuda"),
                     torch.arange(n - 70000, n, device="cuda")])
    cs = codes[idx].cpu().numpy()
    got = vals[idx].cpu().numpy(); want = oracle.hif8_decode(cs)
    ok = ~np.isnan(want)
    assert np.array_equal(np.isnan(got), np.isnan(want))
    assert np.array_equal(got[ok].astype(np.float64), want[ok])
    assert np.array_equal(p[idx].cpu().numpy(), oracle.exp2_code_table()[cs])
