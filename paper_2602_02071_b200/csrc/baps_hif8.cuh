// HiF8 arithmetic for the CUDA path: rounding, code packing/unpacking and the table of
// w0(u) = HiF8(2^HiF8(u)) (Algorithm 1, lines "T in 8-bit" and "P = 2^T in 8-bit"; Algorithm 2).
//
// Blackwell has no HiF8 datatype, so everything here is integer manipulation of fp32 bit
// patterns.  The format keeps 3 mantissa bits for exponents -3..3, 2 bits for |E| in 4..7,
// 1 bit for |E| in 8..15 and none in the denormal range 2^-22..2^-16.  Rounding to nearest with
// ties to the larger magnitude is "add half a step of the binade's grid, truncate, let the
// carry run into the exponent", so the result depends only on sign, exponent and the top four
// mantissa bits of the fp32 input.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace baps {

// Value of HiF8(x) as a float.  +-inf for |x| >= 40960 (midpoint between the largest finite
// value 2^15 and the code position of infinity, 1.5 * 2^15), +0 for |x| < 2^-23, NaN for NaN.
__host__ __device__ __forceinline__ float hif8_round(float x)
{
#ifdef __CUDA_ARCH__
    uint32_t b = __float_as_uint(x);
#else
    uint32_t b; memcpy(&b, &x, 4);
#endif
    const uint32_t s = b & 0x80000000u;
    const uint32_t a = b & 0x7fffffffu;
    uint32_t r;
    if (a >= 0x47200000u) {                 // >= 40960, inf or NaN
        r = (a > 0x7f800000u) ? 0x7fc00000u : (s | 0x7f800000u);
    } else if (a < 0x34000000u) {           // < 2^-23: zero (the format has no negative zero)
        r = 0u;
    } else if (a < 0x34800000u) {           // [2^-23, 2^-22): the neighbours are 0 and 2^-22
        r = s | 0x34800000u;
    } else {
        const int e = (int)(a >> 23) - 127;
        const int ae = e < 0 ? -e : e;
        const int k = (ae <= 3) ? 3 : (ae <= 7) ? 2 : (ae <= 15) ? 1 : 0;
        const uint32_t half = 0x00400000u >> k;
        r = s | ((a + half) & ~((half << 1) - 1u));
    }
#ifdef __CUDA_ARCH__
    return __uint_as_float(r);
#else
    float f; memcpy(&f, &r, 4); return f;
#endif
}

// Pack a float that already is a HiF8 value (output of hif8_round) into its code.
__host__ __device__ __forceinline__ uint8_t hif8_pack(float v)
{
#ifdef __CUDA_ARCH__
    uint32_t b = __float_as_uint(v);
#else
    uint32_t b; memcpy(&b, &v, 4);
#endif
    const uint32_t s = (b >> 31) << 7;
    const uint32_t a = b & 0x7fffffffu;
    if (a > 0x7f800000u) return 0x80;                 // NaN
    if (a == 0u) return 0x00;
    if (a == 0x7f800000u) return (uint8_t)(s | 0x6Fu);
    const int e = (int)(a >> 23) - 127;
    const uint32_t m3 = (a >> 20) & 7u;               // top three mantissa bits
    const uint32_t se = e < 0 ? 1u : 0u;
    const int ae = e < 0 ? -e : e;
    uint32_t c;
    if (e < -15) c = (uint32_t)(e + 23);                               // 0000 mmm (denormal)
    else if (ae == 0) c = 0x08u | m3;                                  // 0001 mmm
    else if (ae == 1) c = 0x10u | (se << 3) | m3;                      // 001 e mmm
    else if (ae <= 3) c = 0x20u | (se << 4) | ((uint32_t)(ae - 2) << 3) | m3;          // 01 ee mmm
    else if (ae <= 7) c = 0x40u | (se << 4) | ((uint32_t)(ae - 4) << 2) | (m3 >> 1);   // 10 eee mm
    else c = 0x60u | (se << 4) | ((uint32_t)(ae - 8) << 1) | (m3 >> 2);                // 11 eeee m
    return (uint8_t)(s | c);
}

__host__ __device__ __forceinline__ uint8_t hif8_encode(float x) { return hif8_pack(hif8_round(x)); }

// Value of a code.
__host__ __device__ __forceinline__ float hif8_unpack(uint8_t code)
{
    const uint32_t s = (uint32_t)(code >> 7) << 31;
    const uint32_t b = code & 0x7Fu;
    uint32_t r;
    if (b == 0u) {
        r = s ? 0x7fc00000u : 0u;
    } else {
        int e; uint32_t m3;                            // mantissa left-aligned to three bits
        if ((b >> 5) == 3u) { e = 8 + (int)((b >> 1) & 7u); if (b & 0x10u) e = -e; m3 = (b & 1u) << 2; }
        else if ((b >> 5) == 2u) { e = 4 + (int)((b >> 2) & 3u); if (b & 0x10u) e = -e; m3 = (b & 3u) << 1; }
        else if ((b >> 5) == 1u) { e = 2 + (int)((b >> 3) & 1u); if (b & 0x10u) e = -e; m3 = b & 7u; }
        else if ((b >> 4) == 1u) { e = (b & 8u) ? -1 : 1; m3 = b & 7u; }
        else if ((b >> 3) == 1u) { e = 0; m3 = b & 7u; }
        else { e = (int)b - 23; m3 = 0u; }
        if (b == 0x6Fu) r = s | 0x7f800000u;
        else r = s | ((uint32_t)(e + 127) << 23) | (m3 << 20);
    }
#ifdef __CUDA_ARCH__
    return __uint_as_float(r);
#else
    float f; memcpy(&f, &r, 4); return f;
#endif
}

// HiF8(2^t) for a HiF8 value t, as a float: the real 2^t (double precision exp2) rounded once.
__device__ __forceinline__ float hif8_exp2_value(float t)
{
    if (t != t) return t;
    double y = exp2((double)t);
    float yf = (y > 3.0e38) ? __uint_as_float(0x7f800000u) : (float)y;
    return hif8_round(yf);
}

// ------------------------------------------------------------------------------------------
// Table of w0(u) = HiF8(2^HiF8(u)) indexed by the top 13 bits of the fp32 pattern of u
// (sign, exponent, four mantissa bits).  Only two index windows matter:
//   negative u with |u| in [2^-6, 32): smaller |u| give 1.0, larger give 0 (clamped ends);
//   positive u in [2^-6, 4): reachable only while the rounded T stays <= lambda <= 3.
// ------------------------------------------------------------------------------------------
constexpr int kLutNegLo = 0x1000 | ((127 - 6) << 4);        // key of -2^-6
constexpr int kLutNegHi = (0x1000 | ((127 + 5) << 4)) - 1;  // last key below -32 ... see below
constexpr int kLutNegN = kLutNegHi - kLutNegLo + 2;         // one extra entry: |u| >= 32 -> 0
constexpr int kLutPosLo = (127 - 6) << 4;                   // key of +2^-6
constexpr int kLutPosHi = ((127 + 2) << 4) - 1;             // last key below +4
constexpr int kLutPosN = kLutPosHi - kLutPosLo + 1;
constexpr int kLutN = kLutNegN + kLutPosN;                  // 177 + 128 entries

// Entry i of the table (device-side build; 2^t in double so that no entry depends on the
// accuracy of the hardware exponential).
__device__ __forceinline__ float w0_table_entry(int i)
{
    uint32_t key;
    if (i < kLutNegN) key = (uint32_t)(kLutNegLo + i);
    else key = (uint32_t)(kLutPosLo + (i - kLutNegN));
    const float u = __uint_as_float(key << 19);
    return hif8_exp2_value(hif8_round(u));
}

// Index of u into the table.
__device__ __forceinline__ int w0_index(float u)
{
    const int key = (int)(__float_as_uint(u) >> 19);
    if (key & 0x1000) return min(max(key, kLutNegLo), kLutNegHi + 1) - kLutNegLo;
    return kLutNegN + min(max(key, kLutPosLo), kLutPosHi) - kLutPosLo;
}

} // namespace baps
