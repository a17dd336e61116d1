"""ctypes front-end of the C oracle (``baps_oracle.c``) -- TEST INFRASTRUCTURE.

Everything numerical lives in the C file, which cites the passages of the paper it follows;
this module only compiles it with gcc, marshals numpy arrays and returns numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "baps_oracle.c")
_LIB = os.path.join(_HERE, "libbaps_oracle.so")

MODE_E2E_HIF8 = 0   # Algorithm 1 with HiF8 roundings
MODE_EXACT = 1      # Eq. (1) in double precision
MODE_EXP2_HIF8 = 2  # Eq. (2) with every power of two through Algorithm 2 ("Exp2 HiF8" setup)
MODE_IDENTITY = 3   # Algorithm 1 with the roundings removed (structure check only)
MODE_EXP2_IDENTITY = 4  # the Exp2 setup with the roundings removed (structure check only)
MODE_EXP2_E4M3 = 5      # comparison setups of Section 4.2: the Exp2 setup with E4M3 in and out,
MODE_EXP2_E5M2 = 6      # ... with E5M2 in and out,
MODE_EXP2_E4M3_E5M2 = 7  # ... with E4M3 arguments and E5M2 results,
MODE_NAIVE_E2E = 8      # and "Naive E2E": scores cast to HiF8 before the max is subtracted

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP) next to its source and return the path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    c_dp = ctypes.POINTER(ctypes.c_double)
    c_fp = ctypes.POINTER(ctypes.c_float)
    c_u8p = ctypes.POINTER(ctypes.c_uint8)
    c_i32p = ctypes.POINTER(ctypes.c_int32)
    lib.baps_oracle_hif8_value.restype = ctypes.c_double
    lib.baps_oracle_hif8_value.argtypes = [ctypes.c_uint8]
    lib.baps_oracle_hif8_encode.restype = None
    lib.baps_oracle_hif8_encode.argtypes = [c_dp, c_u8p, ctypes.c_int64]
    lib.baps_oracle_hif8_decode.restype = None
    lib.baps_oracle_hif8_decode.argtypes = [c_u8p, c_dp, ctypes.c_int64]
    lib.baps_oracle_exp2_code.restype = ctypes.c_uint8
    lib.baps_oracle_exp2_code.argtypes = [ctypes.c_uint8]
    lib.baps_oracle_encode_scalar.restype = ctypes.c_uint8
    lib.baps_oracle_encode_scalar.argtypes = [ctypes.c_double]
    lib.baps_oracle_attention.restype = ctypes.c_int
    lib.baps_oracle_attention.argtypes = [
        c_fp, c_fp, c_fp, c_dp,
        ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
        ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_double, ctypes.c_double,
        c_i32p, ctypes.c_int64, c_dp, c_dp, c_dp, c_dp, c_i32p, c_i32p,
    ]
    lib.baps_oracle_softmax_rows.restype = ctypes.c_int
    lib.baps_oracle_softmax_rows.argtypes = [
        c_fp, c_dp, ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
        ctypes.c_double, c_dp, c_dp,
    ]
    lib.baps_oracle_num_threads.restype = ctypes.c_int
    lib.baps_oracle_softmax_rows_codes.restype = ctypes.c_int
    lib.baps_oracle_softmax_rows_codes.argtypes = [c_fp, c_u8p, c_i32p, c_dp, ctypes.c_int64, ctypes.c_int64,
                                                   ctypes.c_int, ctypes.c_int]
    for fn in (lib.baps_oracle_round_e4m3, lib.baps_oracle_round_e5m2):
        fn.restype = ctypes.c_double
        fn.argtypes = [ctypes.c_double]
    _lib = lib
    return lib


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def num_threads() -> int:
    """Threads the OpenMP loops of the oracle will use."""
    return int(_load().baps_oracle_num_threads())


def hif8_value_table() -> np.ndarray:
    """value(code) for the 256 HiF8 codes (float64; 0x80 is NaN, 0x6F / 0xEF are +-inf)."""
    lib = _load()
    return np.array([lib.baps_oracle_hif8_value(c) for c in range(256)], dtype=np.float64)


def hif8_encode(x) -> np.ndarray:
    """HiF8 code of each element of x (nearest value, ties to the larger magnitude)."""
    x = np.ascontiguousarray(np.asarray(x, dtype=np.float64))
    out = np.empty(x.shape, dtype=np.uint8)
    _load().baps_oracle_hif8_encode(_p(x, ctypes.c_double), _p(out, ctypes.c_uint8), x.size)
    return out


def hif8_decode(codes) -> np.ndarray:
    codes = np.ascontiguousarray(np.asarray(codes, dtype=np.uint8))
    out = np.empty(codes.shape, dtype=np.float64)
    _load().baps_oracle_hif8_decode(_p(codes, ctypes.c_uint8), _p(out, ctypes.c_double), codes.size)
    return out


def exp2_code_table() -> np.ndarray:
    """EXP2_8: code of HiF8(2^value(t)) for every input code t (Algorithm 2)."""
    lib = _load()
    return np.array([lib.baps_oracle_exp2_code(t) for t in range(256)], dtype=np.uint8)


def encode_scalar(y: float) -> int:
    return int(_load().baps_oracle_encode_scalar(float(y)))


def round_e4m3(x) -> np.ndarray:
    """OCP E4M3 rounding (nearest, ties to even, saturating at 448) of each element."""
    lib = _load()
    return np.array([lib.baps_oracle_round_e4m3(float(t)) for t in np.asarray(x, dtype=np.float64).ravel()]).reshape(np.shape(x))


def round_e5m2(x) -> np.ndarray:
    """OCP E5M2 rounding (nearest, ties to even, saturating at 57344) of each element."""
    lib = _load()
    return np.array([lib.baps_oracle_round_e5m2(float(t)) for t in np.asarray(x, dtype=np.float64).ravel()]).reshape(np.shape(x))


def all_tiles(B: int, H: int, S: int, block_q: int) -> np.ndarray:
    """(b, h, i) for every query tile, in [B, H, S / block_q] order."""
    b, h, i = np.meshgrid(np.arange(B), np.arange(H), np.arange(S // block_q), indexing="ij")
    return np.stack([b.ravel(), h.ravel(), i.ravel()], axis=1).astype(np.int32)


@dataclass
class AttentionResult:
    out: np.ndarray          # [n_sel, block_q, D] float64, unrounded O
    row_m: np.ndarray        # [n_sel, block_q] final integer max
    row_d: np.ndarray        # [n_sel, block_q] final denominator
    row_margin: np.ndarray   # [n_sel, block_q] smallest relative distance of a row decision to its boundary
    row_allow: np.ndarray    # [n_sel, block_q] output change bound from near-boundary element roundings
    restarts: np.ndarray     # [n_sel] restarted B1 tiles
    n_tiles: np.ndarray      # [n_sel] key tiles visited
    tiles: np.ndarray        # [n_sel, 3]


def attention(q, k, v, *, causal: bool, block_q: int, block_k: int, lam: int = 1,
              mode: int = MODE_E2E_HIF8, scale: float = 0.0, tiles=None,
              eps_rel: float = 2.0 ** -16, b0_last: bool = False) -> AttentionResult:
    """Attention of q [B,H,S,D] against k, v [B,Hkv,S,D] (float32 arrays holding the inputs
    exactly), for the selected query tiles (default: all).  b0_last: the high-precision set B0 is
    the first and the last visible key tile instead of the first one alone."""
    q = np.ascontiguousarray(np.asarray(q, dtype=np.float32))
    k = np.ascontiguousarray(np.asarray(k, dtype=np.float32))
    v = np.ascontiguousarray(np.asarray(v, dtype=np.float32))
    B, H, S, D = q.shape
    Hkv = k.shape[1]
    assert k.shape == (B, Hkv, S, D) and v.shape == (B, Hkv, S, D)
    if tiles is None:
        tiles = all_tiles(B, H, S, block_q)
    tiles = np.ascontiguousarray(np.asarray(tiles, dtype=np.int32).reshape(-1, 3))
    n = tiles.shape[0]
    out = np.zeros((n, block_q, D), dtype=np.float64)
    row_m = np.zeros((n, block_q)); row_d = np.zeros((n, block_q))
    row_margin = np.full((n, block_q), np.inf); row_allow = np.zeros((n, block_q))
    restarts = np.zeros(n, dtype=np.int32); n_tiles = np.zeros(n, dtype=np.int32)
    dp = ctypes.c_double
    rc = _load().baps_oracle_attention(
        _p(q, ctypes.c_float), _p(k, ctypes.c_float), _p(v, ctypes.c_float), _p(out, dp),
        B, H, Hkv, S, D, int(bool(causal)), block_q, block_k, int(lam), int(mode), int(bool(b0_last)), float(scale),
        float(eps_rel), _p(tiles, ctypes.c_int32), n,
        _p(row_m, dp), _p(row_d, dp), _p(row_margin, dp), _p(row_allow, dp),
        _p(restarts, ctypes.c_int32), _p(n_tiles, ctypes.c_int32))
    if rc != 0:
        raise ValueError("baps_oracle_attention: invalid arguments")
    return AttentionResult(out, row_m, row_d, row_margin, row_allow, restarts, n_tiles, tiles)


def softmax_rows(logits, *, block_k: int, lam: int = 1, identity: bool = False,
                 eps_rel: float = 2.0 ** -16, want_allow: bool = False):
    """Row softmax by Algorithm 1 restricted to single rows.  Returns probs (float64) and,
    if want_allow, also (row_margin, allow)."""
    x = np.ascontiguousarray(np.asarray(logits, dtype=np.float32))
    rows, cols = x.shape
    probs = np.zeros((rows, cols), dtype=np.float64)
    dp = ctypes.c_double
    margin = np.full(rows, np.inf)
    allow = np.zeros((rows, cols)) if want_allow else None
    rc = _load().baps_oracle_softmax_rows(
        _p(x, ctypes.c_float), _p(probs, dp), rows, cols, block_k, int(lam), int(bool(identity)),
        float(eps_rel), _p(margin, dp), _p(allow, dp) if want_allow else None)
    if rc != 0:
        raise ValueError("baps_oracle_softmax_rows: invalid arguments")
    if want_allow:
        return probs, margin, allow
    return probs


def softmax_rows_codes(logits, *, block_k: int, lam: int = 1):
    """Row softmax with 8-bit output: returns (codes uint8 [rows, cols], block_exp int32 [rows, cols /
    block_k], row_d float64 [rows]) with probs = value(codes) * 2^block_exp / row_d.  Decisions are
    taken in single precision, as the CUDA kernel takes them, so that codes compare bit for bit."""
    x = np.ascontiguousarray(np.asarray(logits, dtype=np.float32))
    rows, cols = x.shape
    codes = np.zeros((rows, cols), dtype=np.uint8)
    bexp = np.zeros((rows, cols // block_k), dtype=np.int32)
    d = np.zeros(rows, dtype=np.float64)
    rc = _load().baps_oracle_softmax_rows_codes(_p(x, ctypes.c_float), _p(codes, ctypes.c_uint8),
                                                _p(bexp, ctypes.c_int32), _p(d, ctypes.c_double), rows, cols,
                                                int(block_k), int(lam))
    if rc != 0:
        raise ValueError("baps_oracle_softmax_rows_codes: invalid arguments")
    return codes, bexp, d
