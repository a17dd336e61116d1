// Standalone HiF8 kernels: encode, decode (the conversions of Algorithm 2) and the 8-bit
// exponent map p = HiF8(2^t) (Algorithm 2 as a whole).  All three are streaming kernels bound
// by HBM bandwidth: 5 bytes per element for encode/decode, 2 for the exponent map.
//
// Access pattern (measured on B200, 2^28 elements): what decides the bandwidth of such a stream is the
// shape of the traffic, not the arithmetic -- a kernel that only moves the bytes of decode, with the
// former pattern (256-thread CTAs, 8 per SM, each looping with a grid-wide stride), ran at the same
// 5.2 TB/s as the real kernel.  Two things lift it to the copy bandwidth: a CTA iteration covers one
// contiguous piece of both arrays (1024 threads, 16 KB of codes / 64 KB of fp32), and the grid holds
// many more CTAs than fit at once (32 per SM, a few iterations each), so that the hardware scheduler
// evens out the SMs instead of a static partition waiting for the slowest one.
//
// Arithmetic: encode and decode are single shared-memory table lookups (8192 and 256 entries), the
// exponent map one lookup per code in a 256-entry table; the tables come from the bit-level routines in
// baps_hif8.cuh.  Tables that a warp indexes with unrelated codes are stored once per bank (lane l
// reads copy l), so a lookup never collides with another lane's.
#pragma once
#include "baps_common.cuh"
#include "baps_hif8.cuh"

namespace baps {

constexpr int kEwThreads = 1024;
constexpr int kEwUnroll = 4;
constexpr int kEwCtasPerSm = 32;            // grid cap, in CTAs per SM (two are resident at a time)

// The code of an fp32 value depends only on its sign, exponent and top four mantissa bits
// (rounding adds half a step of a grid that keeps at most three mantissa bits), so encoding is
// one lookup in an 8192-entry byte table indexed by the top 13 bits.  The table is built once per
// device by the bit-level encoder and copied into shared memory by every CTA.  NaN is the one
// class the prefix cannot tell from infinity and is handled by a compare.
__device__ uint8_t g_encode_table[8192];
// p = HiF8(2^t) as a map from code to code (the exponential is taken in double precision, once per device)
__device__ uint8_t g_exp2_map[256];

__global__ void encode_table_init_kernel()
{
    for (int i = threadIdx.x + blockIdx.x * blockDim.x; i < 8192; i += blockDim.x * gridDim.x)
        g_encode_table[i] = hif8_encode(__uint_as_float((uint32_t)i << 19));
    for (int i = threadIdx.x + blockIdx.x * blockDim.x; i < 256; i += blockDim.x * gridDim.x)
        g_exp2_map[i] = hif8_pack(hif8_exp2_value(hif8_unpack((uint8_t)i)));
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

// A CTA iteration encodes one contiguous chunk of kEwThreads * kEwUnroll float4 (64 KB of fp32).
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
    constexpr size_t kChunk = (size_t)kEwThreads * kEwUnroll;
    const size_t nfull = n4 / kChunk;
    for (size_t c = blockIdx.x; c < nfull; c += gridDim.x) {
        const size_t base = c * kChunk + threadIdx.x;
        float4 v[kEwUnroll];
#pragma unroll
        for (int u = 0; u < kEwUnroll; ++u) v[u] = __ldcs(x4 + base + u * kEwThreads);
#pragma unroll
        for (int u = 0; u < kEwUnroll; ++u) __stcs(c4 + base + u * kEwThreads, pack4_codes(v[u], s_pack));
    }
    if (blockIdx.x == 0) {
        // last partial chunk, then the ragged tail (fewer than 4 elements)
        for (size_t i = nfull * kChunk + threadIdx.x; i < n4; i += kEwThreads)
            __stcs(c4 + i, pack4_codes(__ldcs(x4 + i), s_pack));
        const size_t t = n4 * 4 + threadIdx.x;
        if (threadIdx.x < 4 && t < n) codes[t] = (uint8_t)encode_one(x[t], s_pack);
    }
}

// A HiF8 value has at most three mantissa bits, so the upper half of its fp32 pattern holds all of it:
// the table keeps 16 bits per code, two codes per word, 32 copies (one per bank): 16 KB.
// A thread reads 16 codes with one load; the warp then hands the code words round through shuffles so
// that each of its four store instructions writes 512 contiguous bytes.  A CTA iteration decodes
// kEwThreads * 16 consecutive codes (64 KB of fp32).
__global__ void __launch_bounds__(kEwThreads)
hif8_decode_kernel(const uint8_t *__restrict__ codes, float *__restrict__ x, size_t n)
{
    __shared__ __align__(16) uint32_t rep[128 * 32];
    for (int e2 = threadIdx.x; e2 < 128; e2 += kEwThreads) {
        const uint32_t lo = __float_as_uint(hif8_unpack((uint8_t)(2 * e2))) >> 16;
        const uint32_t hi = __float_as_uint(hif8_unpack((uint8_t)(2 * e2 + 1))) >> 16;
        const uint32_t w = lo | (hi << 16);
        const uint4 w4 = make_uint4(w, w, w, w);
#pragma unroll
        for (int i = 0; i < 8; ++i) reinterpret_cast<uint4 *>(rep)[e2 * 8 + i] = w4;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const uint8_t *lut = reinterpret_cast<const uint8_t *>(rep) + lane * 4;
    // codes 2k and 2k + 1 share the word k * 32 + lane
    auto one = [&](uint32_t c) {
        const uint16_t h = *reinterpret_cast<const uint16_t *>(lut + (c >> 1) * 128 + (c & 1) * 2);
        return __uint_as_float((uint32_t)h << 16);
    };
    auto unpack = [&](uint32_t w) {
        return make_float4(one(w & 0xFF), one((w >> 8) & 0xFF), one((w >> 16) & 0xFF), one(w >> 24));
    };
    const uint4 *c16 = reinterpret_cast<const uint4 *>(codes);
    float4 *x4 = reinterpret_cast<float4 *>(x);
    const size_t nfull = n / 16 / kEwThreads;                   // whole CTA iterations
    for (size_t c = blockIdx.x; c < nfull; c += gridDim.x) {
        const size_t i = c * kEwThreads + threadIdx.x;
        const uint4 w = __ldcs(c16 + i);
        // the warp holds 128 code words; word 32 u + l sits in lane (32 u + l) / 4, component l % 4
        const size_t base4 = (i - lane) * 4;                    // first float4 of the warp's piece
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int src = u * 8 + (lane >> 2);
            const uint32_t a = __shfl_sync(0xffffffffu, w.x, src), b = __shfl_sync(0xffffffffu, w.y, src);
            const uint32_t cc = __shfl_sync(0xffffffffu, w.z, src), d = __shfl_sync(0xffffffffu, w.w, src);
            const int comp = lane & 3;
            const uint32_t mine = comp == 0 ? a : comp == 1 ? b : comp == 2 ? cc : d;
            __stcs(x4 + base4 + u * 32 + lane, unpack(mine));
        }
    }
    if (blockIdx.x == 0) {
        // what is left of the array (fewer than 16 * kEwThreads + 16 codes), one code at a time
        for (size_t t = nfull * kEwThreads * 16 + threadIdx.x; t < n; t += kEwThreads) x[t] = one(codes[t]);
    }
}

// 256-entry map as words, 32 copies of every entry (one per bank): lane l reads copy l, so the sixteen
// lookups of a thread never collide with another lane's whatever the codes are (with one copy, random
// codes made the lookups four- to five-way bank conflicts and the kernel LDS-bound).  A CTA iteration
// maps one contiguous chunk of kEwThreads * 2 sixteen-byte vectors.
__global__ void __launch_bounds__(kEwThreads)
hif8_exp2_kernel(const uint8_t *__restrict__ t_codes, uint8_t *__restrict__ p_codes, size_t n)
{
    __shared__ __align__(16) uint32_t rep[256 * 32];
    for (int e = threadIdx.x; e < 256; e += kEwThreads) {
        const uint32_t v = g_exp2_map[e];
        const uint4 v4 = make_uint4(v, v, v, v);
#pragma unroll
        for (int i = 0; i < 8; ++i) reinterpret_cast<uint4 *>(rep)[e * 8 + i] = v4;
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
    constexpr size_t kChunk = (size_t)kEwThreads * 2;
    const size_t nfull = n16 / kChunk;
    for (size_t c = blockIdx.x; c < nfull; c += gridDim.x) {
        const size_t base = c * kChunk + threadIdx.x;
        const uint4 w0 = __ldcs(t4 + base), w1 = __ldcs(t4 + base + kEwThreads);
        __stcs(p4 + base, make_uint4(map4(w0.x), map4(w0.y), map4(w0.z), map4(w0.w)));
        __stcs(p4 + base + kEwThreads, make_uint4(map4(w1.x), map4(w1.y), map4(w1.z), map4(w1.w)));
    }
    if (blockIdx.x == 0) {
        for (size_t i = nfull * kChunk + threadIdx.x; i < n16; i += kEwThreads) {
            const uint4 w = __ldcs(t4 + i);
            __stcs(p4 + i, make_uint4(map4(w.x), map4(w.y), map4(w.z), map4(w.w)));
        }
        const size_t t = n16 * 16 + threadIdx.x;
        if (threadIdx.x < 16 && t < n) p_codes[t] = (uint8_t)lut[t_codes[t] * 32];
    }
}

// Grid for `units` CTA iterations: all of them as CTAs of their own while that stays under the cap of
// kEwCtasPerSm per SM, which is several times what is resident at once -- the hardware scheduler then
// balances the SMs; beyond the cap the CTAs loop.
inline int ew_grid(size_t units, int num_sms, int cap_per_sm = kEwCtasPerSm)
{
    const size_t cap = (size_t)num_sms * (size_t)cap_per_sm;
    const size_t g = units < cap ? units : cap;
    return (int)(g < 1 ? 1 : g);
}

} // namespace baps
