// Standalone HiF8 kernels: encode, decode (the conversions of Algorithm 2) and the 8-bit
// exponent map p = HiF8(2^t) (Algorithm 2 as a whole).  All three are streaming kernels bound
// by HBM bandwidth: 5 bytes per element for encode/decode, 2 for the exponent map.
//
// Access pattern: a thread handles four consecutive elements per step, so that a warp reads
// 512 contiguous bytes of fp32 (one 16-byte load per lane) and writes 128 contiguous bytes of
// codes (one 4-byte store per lane), or the reverse for decode; four such steps are unrolled to
// keep enough bytes in flight.  The grid is a multiple of the SM count and strides over the array.
//
// Arithmetic: encode and decode are single shared-memory table lookups (8192 and 256 entries);
// the tables come from the bit-level routines in baps_hif8.cuh.
#pragma once
#include "baps_common.cuh"
#include "baps_hif8.cuh"

namespace baps {

constexpr int kEwThreads = 256;
constexpr int kEwUnroll = 4;

// The code of an fp32 value depends only on its sign, exponent and top four mantissa bits
// (rounding adds half a step of a grid that keeps at most three mantissa bits), so encoding is
// one lookup in an 8192-entry byte table indexed by the top 13 bits.  The table is built once per
// device by the bit-level encoder and copied into shared memory by every CTA.  NaN is the one
// class the prefix cannot tell from infinity and is handled by a compare.
__device__ uint8_t g_encode_table[8192];

__global__ void encode_table_init_kernel()
{
    for (int i = threadIdx.x + blockIdx.x * blockDim.x; i < 8192; i += blockDim.x * gridDim.x)
        g_encode_table[i] = hif8_encode(__uint_as_float((uint32_t)i << 19));
}

__device__ __forceinline__ uint32_t encode_one(float x, const uint8_t *s_tab)
{
    const uint32_t b = __float_as_uint(x);
    const uint32_t code = s_tab[b >> 19];
    return ((b & 0x7fffffffu) > 0x7f800000u) ? 0x80u : code;
}

__device__ __forceinline__ uint32_t pack4_codes(float4 f, const uint8_t *s_tab)
{
    return encode_one(f.x, s_tab) | (encode_one(f.y, s_tab) << 8) | (encode_one(f.z, s_tab) << 16) |
           (encode_one(f.w, s_tab) << 24);
}

__global__ void __launch_bounds__(kEwThreads)
hif8_encode_kernel(const float *__restrict__ x, uint8_t *__restrict__ codes, size_t n)
{
    __shared__ __align__(16) uint8_t s_pack[8192];
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(g_encode_table);
        uint4 *dst = reinterpret_cast<uint4 *>(s_pack);
        for (int i = threadIdx.x; i < 8192 / 16; i += kEwThreads) dst[i] = src[i];
    }
    __syncthreads();
    const size_t n4 = n / 4;
    const float4 *x4 = reinterpret_cast<const float4 *>(x);
    uint32_t *c4 = reinterpret_cast<uint32_t *>(codes);
    const size_t stride = (size_t)gridDim.x * kEwThreads;
    size_t i = (size_t)blockIdx.x * kEwThreads + threadIdx.x;
    for (; i + (kEwUnroll - 1) * stride < n4; i += kEwUnroll * stride) {
        float4 v[kEwUnroll];
#pragma unroll
        for (int u = 0; u < kEwUnroll; ++u) v[u] = __ldcs(x4 + i + u * stride);
#pragma unroll
        for (int u = 0; u < kEwUnroll; ++u) __stcs(c4 + i + u * stride, pack4_codes(v[u], s_pack));
    }
    for (; i < n4; i += stride) __stcs(c4 + i, pack4_codes(__ldcs(x4 + i), s_pack));
    // ragged tail (fewer than 4 elements)
    if (blockIdx.x == 0 && threadIdx.x < 4) {
        const size_t t = n4 * 4 + threadIdx.x;
        if (t < n) codes[t] = (uint8_t)encode_one(x[t], s_pack);
    }
}

__global__ void __launch_bounds__(kEwThreads)
hif8_decode_kernel(const uint8_t *__restrict__ codes, float *__restrict__ x, size_t n)
{
    // 256 values, 32 copies each (one per bank): lane l reads copy l, so the four lookups of a
    // thread never collide with another lane's whatever the codes are
    __shared__ __align__(16) float rep[256 * 32];
    {
        const float v = hif8_unpack((uint8_t)threadIdx.x);      // blockDim.x == 256
        const float4 v4 = make_float4(v, v, v, v);
#pragma unroll
        for (int i = 0; i < 8; ++i) reinterpret_cast<float4 *>(rep)[threadIdx.x * 8 + i] = v4;
    }
    __syncthreads();
    const float *lut = rep + (threadIdx.x & 31);
    const size_t n4 = n / 4;
    const uint32_t *c4 = reinterpret_cast<const uint32_t *>(codes);
    float4 *x4 = reinterpret_cast<float4 *>(x);
    const size_t stride = (size_t)gridDim.x * kEwThreads;
    size_t i = (size_t)blockIdx.x * kEwThreads + threadIdx.x;
    auto unpack = [&](uint32_t w) {
        return make_float4(lut[(w & 0xFF) * 32], lut[((w >> 8) & 0xFF) * 32], lut[((w >> 16) & 0xFF) * 32],
                           lut[(w >> 24) * 32]);
    };
    for (; i + (kEwUnroll - 1) * stride < n4; i += kEwUnroll * stride) {
        uint32_t w[kEwUnroll];
#pragma unroll
        for (int u = 0; u < kEwUnroll; ++u) w[u] = __ldcs(c4 + i + u * stride);
#pragma unroll
        for (int u = 0; u < kEwUnroll; ++u) __stcs(x4 + i + u * stride, unpack(w[u]));
    }
    for (; i < n4; i += stride) __stcs(x4 + i, unpack(__ldcs(c4 + i)));
    if (blockIdx.x == 0 && threadIdx.x < 4) {
        const size_t t = n4 * 4 + threadIdx.x;
        if (t < n) x[t] = lut[codes[t] * 32];
    }
}

__global__ void __launch_bounds__(kEwThreads)
hif8_exp2_kernel(const uint8_t *__restrict__ t_codes, uint8_t *__restrict__ p_codes, size_t n)
{
    // 256-entry map, 32 copies of every entry (one per bank, a word each): lane l reads copy l, so the
    // sixteen lookups of a thread never collide with another lane's whatever the codes are (with one
    // copy, random codes made the lookups four- to five-way bank conflicts and the kernel LDS-bound)
    __shared__ __align__(16) uint32_t rep[256 * 32];
    {
        const uint32_t v = hif8_pack(hif8_exp2_value(hif8_unpack((uint8_t)threadIdx.x)));   // blockDim.x == 256
        const uint4 v4 = make_uint4(v, v, v, v);
#pragma unroll
        for (int i = 0; i < 8; ++i) reinterpret_cast<uint4 *>(rep)[threadIdx.x * 8 + i] = v4;
    }
    __syncthreads();
    const uint32_t *lut = rep + (threadIdx.x & 31);
    const size_t n16 = n / 16;
    const uint4 *t4 = reinterpret_cast<const uint4 *>(t_codes);
    uint4 *p4 = reinterpret_cast<uint4 *>(p_codes);
    auto map4 = [&](uint32_t w) {
        return lut[(w & 0xFF) * 32] | (lut[((w >> 8) & 0xFF) * 32] << 8) | (lut[((w >> 16) & 0xFF) * 32] << 16) |
               (lut[(w >> 24) * 32] << 24);
    };
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + stride < n16; i += 2 * stride) {
        const uint4 w0 = __ldcs(t4 + i), w1 = __ldcs(t4 + i + stride);
        __stcs(p4 + i, make_uint4(map4(w0.x), map4(w0.y), map4(w0.z), map4(w0.w)));
        __stcs(p4 + i + stride, make_uint4(map4(w1.x), map4(w1.y), map4(w1.z), map4(w1.w)));
    }
    for (; i < n16; i += stride) {
        const uint4 w = __ldcs(t4 + i);
        __stcs(p4 + i, make_uint4(map4(w.x), map4(w.y), map4(w.z), map4(w.w)));
    }
    if (blockIdx.x == 0) {
        const size_t t = n16 * 16 + threadIdx.x;
        if (threadIdx.x < 16 && t < n) p_codes[t] = (uint8_t)lut[t_codes[t] * 32];
    }
}

inline int ew_grid(size_t n, int num_sms)
{
    const size_t want = (n / 4 + kEwThreads - 1) / kEwThreads;
    const size_t cap = (size_t)num_sms * 8;          // 8 resident CTAs of 256 threads per SM
    size_t g = want < cap ? want : cap;
    return (int)(g < 1 ? 1 : g);
}

} // namespace baps
