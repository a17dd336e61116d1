"""Thin ctypes binding over the C ABI in ``include/baps.h``.

Argument marshalling only: every function takes torch CUDA tensors (used purely as device
buffers), passes their pointers and the current CUDA stream to the entry point of the same
name, and raises ``BapsError`` on a non-zero status.  Nothing here computes: if ``libbaps.so``
is missing the import of the library fails loudly -- there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbaps.so")

BAPS_OK = 0
MODE_E2E_HIF8 = 0
MODE_EXACT = 1
MODE_EXP2_HIF8 = 2
DTYPE_BF16 = 0
DTYPE_F32 = 1

EXPORTS = [
    "baps_hif8_encode", "baps_hif8_decode", "baps_exp2_hif8", "baps_softmax_rows", "baps_softmax_rows_codes",
    "baps_attention_fwd", "baps_attention_fwd_f32", "baps_attention_fwd_ex", "baps_attention_fwd_fp8",
    "baps_attention_restart_rates", "baps_attention_restart_rates_static",
    "baps_status_string", "baps_poll_async_error", "baps_launch_count",
]


class BapsError(RuntimeError):
    def __init__(self, name: str, status: int, text: str):
        super().__init__(f"{name} failed: {text} ({status})")
        self.status = status


class _Opts(ctypes.Structure):
    _fields_ = [("lam", ctypes.c_int), ("mode", ctypes.c_int), ("scale", ctypes.c_float),
                ("b0_last", ctypes.c_int)]


class _Stats(ctypes.Structure):
    _fields_ = [("row_m", ctypes.c_void_p), ("row_d", ctypes.c_void_p),
                ("restarts", ctypes.c_void_p), ("out_f32", ctypes.c_void_p)]


_lib = None


def load() -> ctypes.CDLL:
    """Load ``libbaps.so`` (built by ``paper_2602_02071_b200.build``); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} not found: build it with `python -m paper_2602_02071_b200.build` "
            "(there is no non-CUDA fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i, i64, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t
    lib.baps_hif8_encode.argtypes = [vp, vp, sz, vp]
    lib.baps_hif8_decode.argtypes = [vp, vp, sz, vp]
    lib.baps_exp2_hif8.argtypes = [vp, vp, sz, vp]
    lib.baps_softmax_rows.argtypes = [vp, vp, i64, i64, i, vp]
    lib.baps_attention_fwd.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, i, vp]
    lib.baps_attention_fwd_f32.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, i, vp]
    lib.baps_attention_fwd_ex.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, i, i,
                                          ctypes.POINTER(_Opts), ctypes.POINTER(_Stats), vp]
    lib.baps_attention_restart_rates.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, i, i, vp, sz, vp, vp]
    lib.baps_attention_restart_rates_static.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, i, i, vp, vp]
    lib.baps_softmax_rows_codes.argtypes = [vp, vp, vp, vp, i64, i64, i, vp]
    lib.baps_attention_fwd_fp8.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, i, i, i,
                                           ctypes.POINTER(_Opts), ctypes.POINTER(_Stats), vp]
    for n in EXPORTS[:11]:
        getattr(lib, n).restype = i
    lib.baps_status_string.argtypes = [i]
    lib.baps_status_string.restype = ctypes.c_char_p
    lib.baps_poll_async_error.argtypes = [vp]
    lib.baps_poll_async_error.restype = i
    lib.baps_launch_count.argtypes = []
    lib.baps_launch_count.restype = i64
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().baps_status_string(int(status)).decode()


def _check(name: str, status: int):
    if status != BAPS_OK:
        raise BapsError(name, status, status_string(status))


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _dev(t: torch.Tensor, dtype, name: str):
    if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise ValueError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t


def launch_count() -> int:
    return int(load().baps_launch_count())


def poll_async_error() -> None:
    _check("baps_poll_async_error", load().baps_poll_async_error(_stream()))


def baps_hif8_encode(x: torch.Tensor, codes: Optional[torch.Tensor] = None) -> torch.Tensor:
    _dev(x, torch.float32, "x")
    if codes is None:
        codes = torch.empty(x.shape, dtype=torch.uint8, device=x.device)
    _dev(codes, torch.uint8, "codes")
    _check("baps_hif8_encode", load().baps_hif8_encode(_ptr(x), _ptr(codes), x.numel(), _stream()))
    return codes


def baps_hif8_decode(codes: torch.Tensor, x: Optional[torch.Tensor] = None) -> torch.Tensor:
    _dev(codes, torch.uint8, "codes")
    if x is None:
        x = torch.empty(codes.shape, dtype=torch.float32, device=codes.device)
    _dev(x, torch.float32, "x")
    _check("baps_hif8_decode", load().baps_hif8_decode(_ptr(codes), _ptr(x), codes.numel(), _stream()))
    return x


def baps_exp2_hif8(t_codes: torch.Tensor, p_codes: Optional[torch.Tensor] = None) -> torch.Tensor:
    _dev(t_codes, torch.uint8, "t_codes")
    if p_codes is None:
        p_codes = torch.empty_like(t_codes)
    _dev(p_codes, torch.uint8, "p_codes")
    _check("baps_exp2_hif8", load().baps_exp2_hif8(_ptr(t_codes), _ptr(p_codes), t_codes.numel(), _stream()))
    return p_codes


def baps_softmax_rows(logits: torch.Tensor, block_k: int = 128,
                      probs: Optional[torch.Tensor] = None) -> torch.Tensor:
    _dev(logits, torch.float32, "logits")
    if logits.dim() != 2:
        raise ValueError("logits must be [rows, cols]")
    if probs is None:
        probs = torch.empty_like(logits)
    _dev(probs, torch.float32, "probs")
    rows, cols = logits.shape
    _check("baps_softmax_rows",
           load().baps_softmax_rows(_ptr(logits), _ptr(probs), rows, cols, int(block_k), _stream()))
    return probs


def baps_softmax_rows_codes(logits: torch.Tensor, block_k: int = 128):
    """Row softmax with 8-bit output: returns (codes uint8 [rows, cols], block_exp int32 [rows, cols /
    block_k], row_d float32 [rows]); probs = value(codes) * 2^block_exp / row_d."""
    _dev(logits, torch.float32, "logits")
    if logits.dim() != 2:
        raise ValueError("logits must be [rows, cols]")
    rows, cols = logits.shape
    codes = torch.empty((rows, cols), dtype=torch.uint8, device=logits.device)
    bexp = torch.empty((rows, cols // int(block_k)), dtype=torch.int32, device=logits.device)
    d = torch.empty(rows, dtype=torch.float32, device=logits.device)
    _check("baps_softmax_rows_codes",
           load().baps_softmax_rows_codes(_ptr(logits), _ptr(codes), _ptr(bexp), _ptr(d), rows, cols, int(block_k),
                                          _stream()))
    return codes, bexp, d


def _attn_shapes(q, k, v):
    if q.dim() != 4 or k.dim() != 4 or v.shape != k.shape:
        raise ValueError("q must be [B,H,S,D]; k, v [B,Hkv,S,D]")
    B, H, S, D = q.shape
    if k.shape[0] != B or k.shape[2] != S or k.shape[3] != D:
        raise ValueError("k/v shape does not match q")
    return B, H, k.shape[1], S, D


def baps_attention_fwd(q, k, v, *, causal: bool, block_q: int = 128, block_k: int = 128,
                       out: Optional[torch.Tensor] = None) -> torch.Tensor:
    for t, n in ((q, "q"), (k, "k"), (v, "v")):
        _dev(t, torch.bfloat16, n)
    B, H, Hkv, S, D = _attn_shapes(q, k, v)
    if out is None:
        out = torch.empty_like(q)
    _dev(out, torch.bfloat16, "out")
    _check("baps_attention_fwd",
           load().baps_attention_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, Hkv, S, D,
                                     int(bool(causal)), int(block_q), int(block_k), _stream()))
    return out


def baps_attention_fwd_f32(q, k, v, *, causal: bool, block_q: int = 64, block_k: int = 64,
                           out: Optional[torch.Tensor] = None) -> torch.Tensor:
    for t, n in ((q, "q"), (k, "k"), (v, "v")):
        _dev(t, torch.float32, n)
    B, H, Hkv, S, D = _attn_shapes(q, k, v)
    if out is None:
        out = torch.empty_like(q)
    _dev(out, torch.float32, "out")
    _check("baps_attention_fwd_f32",
           load().baps_attention_fwd_f32(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, Hkv, S, D,
                                         int(bool(causal)), int(block_q), int(block_k), _stream()))
    return out


@dataclass
class AttentionStats:
    out: Optional[torch.Tensor]
    out_f32: Optional[torch.Tensor]
    row_m: Optional[torch.Tensor]
    row_d: Optional[torch.Tensor]
    restarts: Optional[torch.Tensor]


def baps_attention_fwd_ex(q, k, v, *, causal: bool, block_q: int, block_k: int, lam: int = 1,
                          mode: int = MODE_E2E_HIF8, scale: float = 0.0, want_stats: bool = True,
                          out: Optional[torch.Tensor] = None, b0_last: bool = False) -> AttentionStats:
    """Extended call: options plus optional statistics buffers (allocated here with torch and
    handed to the library as plain device pointers)."""
    if q.dtype == torch.bfloat16:
        dtype = DTYPE_BF16
    elif q.dtype == torch.float32:
        dtype = DTYPE_F32
    else:
        raise ValueError("q must be bfloat16 or float32")
    for t, n in ((q, "q"), (k, "k"), (v, "v")):
        _dev(t, q.dtype, n)
    B, H, Hkv, S, D = _attn_shapes(q, k, v)
    if out is None:
        out = torch.empty_like(q)
    st = AttentionStats(out, None, None, None, None)
    cs = _Stats(None, None, None, None)
    if want_stats:
        st.out_f32 = torch.empty(q.shape, dtype=torch.float32, device=q.device)
        st.row_m = torch.empty((B, H, S), dtype=torch.float32, device=q.device)
        st.row_d = torch.empty((B, H, S), dtype=torch.float32, device=q.device)
        st.restarts = torch.zeros((B, H, S // block_q), dtype=torch.int32, device=q.device)
        cs = _Stats(_ptr(st.row_m), _ptr(st.row_d), _ptr(st.restarts), _ptr(st.out_f32))
    opts = _Opts(int(lam), int(mode), float(scale), int(bool(b0_last)))
    _check("baps_attention_fwd_ex",
           load().baps_attention_fwd_ex(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, Hkv, S, D,
                                        int(bool(causal)), int(block_q), int(block_k), dtype,
                                        ctypes.byref(opts), ctypes.byref(cs), _stream()))
    return st


def baps_attention_fwd_fp8(q8, k8, v, q_scale, k_scale, *, causal: bool, lam: int = 1, mode: int = MODE_E2E_HIF8,
                           scale: float = 0.0, want_stats: bool = True, out: Optional[torch.Tensor] = None,
                           b0_last: bool = False) -> AttentionStats:
    """Attention with Q and K given as E4M3 codes (uint8 or torch.float8_e4m3fn tensors) and one
    power-of-two dequantisation scale per 128-row tile (float32 [B,H,S/128] / [B,Hkv,S/128])."""
    q8 = q8.view(torch.uint8) if q8.dtype != torch.uint8 else q8
    k8 = k8.view(torch.uint8) if k8.dtype != torch.uint8 else k8
    _dev(q8, torch.uint8, "q8"); _dev(k8, torch.uint8, "k8"); _dev(v, torch.bfloat16, "v")
    _dev(q_scale, torch.float32, "q_scale"); _dev(k_scale, torch.float32, "k_scale")
    B, H, Hkv, S, D = _attn_shapes(q8, k8, v)
    if q_scale.shape != (B, H, S // 128) or k_scale.shape != (B, Hkv, S // 128):
        raise ValueError("q_scale must be [B,H,S/128], k_scale [B,Hkv,S/128]")
    if out is None:
        out = torch.empty((B, H, S, D), dtype=torch.bfloat16, device=v.device)
    st = AttentionStats(out, None, None, None, None)
    cs = _Stats(None, None, None, None)
    if want_stats:
        st.out_f32 = torch.empty((B, H, S, D), dtype=torch.float32, device=v.device)
        st.row_m = torch.empty((B, H, S), dtype=torch.float32, device=v.device)
        st.row_d = torch.empty((B, H, S), dtype=torch.float32, device=v.device)
        st.restarts = torch.zeros((B, H, S // 128), dtype=torch.int32, device=v.device)
        cs = _Stats(_ptr(st.row_m), _ptr(st.row_d), _ptr(st.restarts), _ptr(st.out_f32))
    opts = _Opts(int(lam), int(mode), float(scale), int(bool(b0_last)))
    _check("baps_attention_fwd_fp8",
           load().baps_attention_fwd_fp8(_ptr(q8), _ptr(k8), _ptr(v), _ptr(out), _ptr(q_scale), _ptr(k_scale),
                                         B, H, Hkv, S, D, int(bool(causal)), 128, 128,
                                         ctypes.byref(opts), ctypes.byref(cs), _stream()))
    return st


def baps_attention_restart_rates(q, k, v, *, causal: bool, lam: int = 1, block_q: int = 128,
                                 block_k: int = 128, out: Optional[torch.Tensor] = None,
                                 scratch: Optional[torch.Tensor] = None):
    """Attention output plus the restart rates of Table 4: returns (out, rates) with rates a CUDA
    float tensor [ARR, PRR].  ``scratch`` (int32, at least B*H*S/128 entries) holds the
    per-query-tile counters between the two kernels; it is allocated here if not given."""
    for t, n in ((q, "q"), (k, "k"), (v, "v")):
        _dev(t, torch.bfloat16, n)
    B, H, Hkv, S, D = _attn_shapes(q, k, v)
    if out is None:
        out = torch.empty_like(q)
    if scratch is None:
        scratch = torch.empty(B * H * (S // 128), dtype=torch.int32, device=q.device)
    _dev(scratch, torch.int32, "scratch")
    rates = torch.empty(2, dtype=torch.float32, device=q.device)
    _check("baps_attention_restart_rates",
           load().baps_attention_restart_rates(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, Hkv, S, D,
                                               int(bool(causal)), int(block_q), int(block_k), int(lam),
                                               _ptr(scratch), scratch.numel(), _ptr(rates), _stream()))
    return out, rates


STATIC_SCRATCH_ENTRIES = 262144


def baps_attention_restart_rates_static(q, k, v, *, causal: bool, out: torch.Tensor, rates: torch.Tensor,
                                        lam: int = 1, block_q: int = 128, block_k: int = 128) -> None:
    """Restart rates for callers that cannot allocate: same results as
    ``baps_attention_restart_rates`` but the counters live in an array built into the library.
    Every buffer, including ``out`` (bf16, shape of q) and ``rates`` (float32[2]), comes from the
    caller; neither this wrapper nor the entry point allocates.  Raises ``BapsError`` with
    BAPS_ERR_SCRATCH_LIMIT when B*H*S/128 exceeds ``STATIC_SCRATCH_ENTRIES``.  Calls share the
    built-in array: do not let two of them overlap on the GPU."""
    for t, n in ((q, "q"), (k, "k"), (v, "v"), (out, "out")):
        _dev(t, torch.bfloat16, n)
    _dev(rates, torch.float32, "rates")
    B, H, Hkv, S, D = _attn_shapes(q, k, v)
    _check("baps_attention_restart_rates_static",
           load().baps_attention_restart_rates_static(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, Hkv, S, D,
                                                      int(bool(causal)), int(block_q), int(block_k), int(lam),
                                                      _ptr(rates), _stream()))
