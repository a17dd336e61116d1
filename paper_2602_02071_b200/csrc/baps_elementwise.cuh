// Standalone HiF8 kernels: encode, decode (the conversions of Algorithm 2) and the 8-bit
// exponent map p = HiF8(2^t) (Algorithm 2 as a whole).  All three are streaming kernels bound
// by HBM bandwidth: 5 bytes per element for encode/decode, 2 for the exponent map.  Each
// thread moves 16 elements per step with 16-byte accesses; the grid is a multiple of the SM
// count and strides over the array.
#pragma once
#include "baps_common.cuh"
#include "baps_hif8.cuh"

namespace baps {

constexpr int kEwThreads = 256;

__device__ __forceinline__ uint32_t pack4_codes(float4 f)
{
    return (uint32_t)hif8_encode(f.x) | ((uint32_t)hif8_encode(f.y) << 8) |
           ((uint32_t)hif8_encode(f.z) << 16) | ((uint32_t)hif8_encode(f.w) << 24);
}

__global__ void __launch_bounds__(kEwThreads)
hif8_encode_kernel(const float *__restrict__ x, uint8_t *__restrict__ codes, size_t n)
{
    const size_t n16 = n / 16;
    const float4 *x4 = reinterpret_cast<const float4 *>(x);
    uint4 *c4 = reinterpret_cast<uint4 *>(codes);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16;
         i += (size_t)gridDim.x * blockDim.x) {
        const float4 a = __ldcs(x4 + 4 * i), b = __ldcs(x4 + 4 * i + 1);
        const float4 c = __ldcs(x4 + 4 * i + 2), d = __ldcs(x4 + 4 * i + 3);
        uint4 o;
        o.x = pack4_codes(a); o.y = pack4_codes(b); o.z = pack4_codes(c); o.w = pack4_codes(d);
        __stcs(c4 + i, o);
    }
    // ragged tail (fewer than 16 elements)
    if (blockIdx.x == 0) {
        const size_t t = n16 * 16 + threadIdx.x;
        if (threadIdx.x < 16 && t < n) codes[t] = hif8_encode(x[t]);
    }
}

__device__ __forceinline__ float4 unpack4_codes(uint32_t w)
{
    return make_float4(hif8_unpack((uint8_t)(w & 0xFF)), hif8_unpack((uint8_t)((w >> 8) & 0xFF)),
                       hif8_unpack((uint8_t)((w >> 16) & 0xFF)), hif8_unpack((uint8_t)(w >> 24)));
}

__global__ void __launch_bounds__(kEwThreads)
hif8_decode_kernel(const uint8_t *__restrict__ codes, float *__restrict__ x, size_t n)
{
    __shared__ float lut[256];
    lut[threadIdx.x] = hif8_unpack((uint8_t)threadIdx.x);      // blockDim.x == 256
    __syncthreads();
    const size_t n16 = n / 16;
    const uint4 *c4 = reinterpret_cast<const uint4 *>(codes);
    float4 *x4 = reinterpret_cast<float4 *>(x);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16;
         i += (size_t)gridDim.x * blockDim.x) {
        const uint4 w = __ldcs(c4 + i);
        const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float4 f = make_float4(lut[ws[j] & 0xFF], lut[(ws[j] >> 8) & 0xFF],
                                   lut[(ws[j] >> 16) & 0xFF], lut[ws[j] >> 24]);
            __stcs(x4 + 4 * i + j, f);
        }
    }
    if (blockIdx.x == 0) {
        const size_t t = n16 * 16 + threadIdx.x;
        if (threadIdx.x < 16 && t < n) x[t] = lut[codes[t]];
    }
}

__global__ void __launch_bounds__(kEwThreads)
hif8_exp2_kernel(const uint8_t *__restrict__ t_codes, uint8_t *__restrict__ p_codes, size_t n)
{
    // 256-entry map, one word per entry so that a lookup never splits a bank word
    __shared__ uint32_t lut[256];
    lut[threadIdx.x] = hif8_pack(hif8_exp2_value(hif8_unpack((uint8_t)threadIdx.x)));
    __syncthreads();
    const size_t n16 = n / 16;
    const uint4 *t4 = reinterpret_cast<const uint4 *>(t_codes);
    uint4 *p4 = reinterpret_cast<uint4 *>(p_codes);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16;
         i += (size_t)gridDim.x * blockDim.x) {
        const uint4 w = __ldcs(t4 + i);
        const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            o[j] = lut[ws[j] & 0xFF] | (lut[(ws[j] >> 8) & 0xFF] << 8) |
                   (lut[(ws[j] >> 16) & 0xFF] << 16) | (lut[ws[j] >> 24] << 24);
        __stcs(p4 + i, make_uint4(o[0], o[1], o[2], o[3]));
    }
    if (blockIdx.x == 0) {
        const size_t t = n16 * 16 + threadIdx.x;
        if (threadIdx.x < 16 && t < n) p_codes[t] = (uint8_t)lut[t_codes[t]];
    }
}

inline int ew_grid(size_t n, int num_sms)
{
    const size_t want = (n / 16 + kEwThreads - 1) / kEwThreads;
    const size_t cap = (size_t)num_sms * 8;          // 8 resident CTAs of 256 threads per SM
    size_t g = want < cap ? want : cap;
    return (int)(g < 1 ? 1 : g);
}

} // namespace baps
