// Fused BAPS attention forward on the 5th-generation tensor cores (tcgen05, sm_100a).
//
// One CTA owns two consecutive 128-row query tiles of one (batch, head) and walks the key
// tiles in increasing order (Algorithm 1: tile 0 is the high-precision set B0, all later
// tiles are 8-bit tiles).  Roles, by warp (640 threads):
//   warps 0-7 / 8-15  softmax warps of query tile 0 / 1.  A row of the 128 x 128 score tile is
//                     shared by two threads: warp w handles rows 32*(w%4) .. +31 (its TMEM
//                     lanes) and the 64 key columns of half (w/4)%2.  Per key tile: half-row
//                     maximum, exchange with the partner thread through shared memory, decide
//                     (B0 / restart / plain), form the weights
//                     w = HiF8(2^HiF8(S*c - m~)) * 2^-delta through a bank-replicated table
//                     indexed by the top bits of the fp32 pattern, write them to TMEM as bf16
//                     (exactly representable) over columns of S the thread has already read.
//                     Four softmax warps per scheduler hide TMEM and table latencies.
//   warp 16           TMA producer: Q tiles once, then K_0, V_0, K_1, V_1, ... through a ring.
//   warp 17           MMA issuer: S_t = Q_t K_j^T (operands in shared memory, 128-byte swizzle)
//                     and O_t += P_t V_j (P from TMEM, V as an MN-major shared operand), ordered
//                     PV_0(j), QK_0(j+1), PV_1(j), QK_1(j+1) so that one tile's softmax overlaps
//                     the other tile's tensor work.  (Warps 18-19 idle: the fifth warpgroup
//                     exists so that its registers can be handed to the softmax warps.)
// TMEM (512 columns): S_0 | S_1 | O_0 | O_1, 128 columns each (64 for O when D = 64).  The bf16
// weights of key half h overwrite columns [64h, 64h + 32) of the tile's S region.
// Every wait on an mbarrier is bounded; on expiry the CTA raises an abort flag, records a code
// in the library's status word and all roles fall through to the common teardown.
#pragma once
#include <cuda_bf16.h>
#include "baps_common.cuh"
#include "baps_hif8.cuh"
#include "baps_sm100.cuh"
#include "baps_tma_host.cuh"

#ifndef BAPS_WAIT_FLAG
#define BAPS_WAIT_FLAG mbar_wait_poll<0>
#endif
#ifndef BAPS_WAIT_PAIR
#define BAPS_WAIT_PAIR mbar_wait_poll<0>
#endif

namespace baps {

// w0 table in global memory, filled once per device by w0_table_init_kernel.
__device__ float g_w0_table[kLutN];

__global__ void w0_table_init_kernel()
{
    for (int i = threadIdx.x; i < kLutN; i += blockDim.x) g_w0_table[i] = w0_table_entry(i);
}

#ifdef BAPS_TRACE
// developer switch: clock64() stamps of CTA 0: [group][tile][warp-in-group][slot]
__device__ long long g_trace[2 * 512 * 4 * 4];
__device__ long long g_trace_mma[2 * 512 * 2];
#endif

struct AttnTcParams {
    __nv_bfloat16 *out;       // [B,H,S,D] or null
    float *out_f32;           // optional
    float *row_m, *row_d;     // optional [B,H,S]
    int32_t *restarts;        // optional [B,H,S/128]
    int B, H, Hkv, S, causal, lambda, mode;
    float c;                  // log2(e) * scale
    int nq, npairs;
};

constexpr int kTcThreads = 640;
constexpr int kTcSoftmaxWarps = 16;
constexpr int kLutRepEntries = 16 + kLutNegN;              // keys 0 .. 192, 32 copies each
constexpr int kLutRepBytes = kLutRepEntries * 128;

template <int D>
struct TcLayout {
    static constexpr int kTileBytes = 128 * D * 2;
    static constexpr int kStages = (D == 128) ? 4 : 8;
    static constexpr int kQOff = 0;
    static constexpr int kKvOff = 2 * kTileBytes;
    static constexpr int kLutRepOff = kKvOff + kStages * kTileBytes;
    static constexpr int kLutFullOff = kLutRepOff + kLutRepBytes;
    static constexpr int kBarOff = (kLutFullOff + kLutN * 4 + 15) & ~15;
    // barriers: q_full, s_full[2], p_full[2], o_full[2], flag[2][2], pair[8], p_half[2], kv_full[S], kv_empty[S]
    static constexpr int kNumBars = 1 + 2 + 2 + 2 + 4 + 8 + 2 + 2 * kStages;
    static constexpr int kFlagOff = kBarOff + kNumBars * 8;          // int flags[2][2][4]
    static constexpr int kXchgOff = kFlagOff + 16 * 4;               // float xchg[2][128][2]
    static constexpr int kMiscOff = kXchgOff + 2 * 128 * 2 * 4;      // tmem base, abort
    static constexpr int kTotal = kMiscOff + 16;
    static constexpr int kDynBytes = kTotal + 1024;                  // slack for 1024-byte alignment
};

__device__ __forceinline__ float lds_f32(uint32_t addr)
{
    float v;
    asm("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float mul_ftz(float a, float b)
{
    float d;
    asm("mul.rn.ftz.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}
// Packed pairs of fp32 (sm_100 FFMA2 / FADD2): one instruction for two elements.
__device__ __forceinline__ uint64_t pack2(float lo, float hi)
{
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t fma2_ftz(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.ftz.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
// 2^k for an integer-valued k (exact); 0 below the normal range, saturating far above it
__device__ __forceinline__ float pow2_int(float k)
{
    const int e = 127 + (int)k;
    return e > 0 ? __int_as_float(min(e, 254) << 23) : 0.f;
}

// ---- fast path -------------------------------------------------------------------------------
// Weights of 16 columns when every T = S*c - mref of the row is <= 0 (a plain 8-bit tile whose
// row maximum did not exceed the running max, or a restarted tile).
//   x   = -T * 2^-120, one packed FMA per two columns with flush-to-zero: x = +0 for
//         |T| < 2^-6 (weight 1), otherwise a normal number with biased exponent >= 1
//   key = min(bits(x) >> 19, 192): exponent and top four mantissa bits (what HiF8 rounding with
//         ties to the larger magnitude depends on); 192 stands for |T| >= 32 (weight 0) and is
//         also where a positive T lands (sign bit set) -- those entries are redone by the caller
//   w   = table[key], 32 copies per entry, one per bank: no conflicts
// The weights are exactly representable in bf16; the power-of-two factor 2^e (e >= 0) that
// expresses them against the accumulators' reference max is added to the packed exponents.
// Unscaled weights are summed pairwise (packed adds).
// kTwoStep (the Exp2 setup, whose running max is not an integer and may be smaller than 2^-6, too
// small to survive the 2^-120 scaling): T = S*c - m by a plain packed FMA (cn2 = c, mn2 = -m),
// then x = T * -2^-120 + 0 with flush-to-zero; the +0 addend turns a cancelled T into +0.
template <bool kTwoStep>
__device__ __forceinline__ void fast16(const uint32_t (&r)[16], uint32_t (&pk)[8], uint64_t cn2, uint64_t mn2,
                                       uint32_t escale, uint32_t tb, uint64_t &s01, uint64_t &s23)
{
    uint32_t a[16];
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
        float x0, x1;
        if constexpr (kTwoStep) {
            const uint64_t t2 = fma2(pack2(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), cn2, mn2);
            unpack2(fma2_ftz(t2, pack2(-7.52316384526264e-37f, -7.52316384526264e-37f), 0ull), x0, x1);
        } else {
            unpack2(fma2_ftz(pack2(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), cn2, mn2), x0, x1);
        }
        a[i] = min(__float_as_uint(x0) >> 19, 192u) * 128u + tb;
        a[i + 1] = min(__float_as_uint(x1) >> 19, 192u) * 128u + tb;
    }
    float w[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) w[i] = lds_f32(a[i]);
#pragma unroll
    for (int i = 0; i < 16; i += 4) {
        s01 = add2(s01, pack2(w[i], w[i + 1]));
        s23 = add2(s23, pack2(w[i + 2], w[i + 3]));
        pk[i >> 1] = pack_bf16x2(w[i], w[i + 1]) + escale;
        pk[(i >> 1) + 1] = pack_bf16x2(w[i + 2], w[i + 3]) + escale;
    }
}

// Eight columns redone with the full, sign-aware table (rows whose maximum rose above the
// running max in a tile that was not restarted have a few positive T; the fast path gives
// those weight 0).  Overwrites four packed registers and returns the amount to add to the sum.
__device__ __forceinline__ float fix8(const uint32_t *x, uint32_t *pk4, float c, float mref, uint32_t escale,
                                      uint32_t lut_full)
{
    float add = 0.f;
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
        const float u0 = fmaf(__uint_as_float(x[i]), c, -mref);
        const float u1 = fmaf(__uint_as_float(x[i + 1]), c, -mref);
        const float w0 = lds_f32(lut_full + 4u * (uint32_t)w0_index(u0));
        const float w1 = lds_f32(lut_full + 4u * (uint32_t)w0_index(u1));
        // the fast path counted 0 for every T > 0 and the same value otherwise
        if (u0 > 0.f) add += w0;
        if (u1 > 0.f) add += w1;
        pk4[i >> 1] = pack_bf16x2(w0, w1) + escale;
    }
    return add;
}

// High-precision tile (B0, or every tile in the exact mode): P = 2^(S*c - mref) in fp32, rounded
// to bf16 for the tensor core; the row sum uses the rounded values so that numerator and
// denominator see the same weights.  Masked entries arrive as -inf and give 0.
__device__ __forceinline__ float hp16(const uint32_t (&r)[16], uint32_t (&pk)[8], float c, float mref)
{
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
        const float u0 = fmaf(__uint_as_float(r[i]), c, -mref);
        const float u1 = fmaf(__uint_as_float(r[i + 1]), c, -mref);
        const uint32_t p = pack_bf16x2(ex2_approx(u0), ex2_approx(u1));
        s0 += __uint_as_float(p << 16);
        s1 += __uint_as_float(p & 0xFFFF0000u);
        pk[i >> 1] = p;
    }
    return s0 + s1;
}

__device__ __forceinline__ float max8(const uint32_t *x)
{
    return max3(max3(__uint_as_float(x[0]), __uint_as_float(x[1]), __uint_as_float(x[2])),
                max3(__uint_as_float(x[3]), __uint_as_float(x[4]), __uint_as_float(x[5])),
                fmaxf(__uint_as_float(x[6]), __uint_as_float(x[7])));
}

// kExp2 selects the "Exp2 HiF8" setup of Section 4.1 (Eq. (2) with a real-valued max, weights and
// rescale factor through the 8-bit exponent table); otherwise Algorithm 1 or the exact mode.
template <int D, bool kExp2>
__global__ void __launch_bounds__(kTcThreads, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mk,
                    const __grid_constant__ CUtensorMap mv, const AttnTcParams p)
{
    using namespace sm100;
    using L = TcLayout<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + L::kBarOff;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    constexpr int BQ = 0, BS = 1, BP = 3, BO = 5, BF = 7, BX = 11, BPA = 19, BKF = 21, BKE = 21 + L::kStages;
    int *s_flags = reinterpret_cast<int *>(smem + L::kFlagOff);
    volatile float *s_xchg = reinterpret_cast<volatile float *>(smem + L::kXchgOff);
    uint32_t *s_tmem = reinterpret_cast<uint32_t *>(smem + L::kMiscOff);
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + L::kMiscOff + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // ---- work assignment: heavy (late) query tiles first; the g query heads of one kv head adjacent
    const int gsz = p.H / p.Hkv;
    int idx = blockIdx.x;
    const int gi = idx % gsz; idx /= gsz;
    const int hk = idx % p.Hkv; idx /= p.Hkv;
    const int b = idx % p.B; idx /= p.B;
    const int pair = p.npairs - 1 - idx;
    const int h = hk * gsz + gi;
    const int nk = p.S / 128;
    int jm[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int qi = 2 * pair + t;
        jm[t] = (qi < p.nq) ? (p.causal ? qi + 1 : nk) : 0;
    }
    const int J = jm[0] > jm[1] ? jm[0] : jm[1];
    const int q_row0 = (b * p.H + h) * p.S + 2 * pair * 128;        // row in the [B*H*S, D] view
    const int kv_row0 = (b * p.Hkv + hk) * p.S;

    // ---- setup --------------------------------------------------------------------------------
    if (tid == 0) {
        mbar_init(bar(BQ), 1);
        for (int t = 0; t < 2; ++t) {
            mbar_init(bar(BS + t), 1);
            mbar_init(bar(BP + t), 256);
            mbar_init(bar(BPA + t), 256);
            mbar_init(bar(BO + t), 1);
            mbar_init(bar(BF + 2 * t), 4);
            mbar_init(bar(BF + 2 * t + 1), 4);
        }
        for (int i = 0; i < 8; ++i) mbar_init(bar(BX + i), 64);
        for (int s = 0; s < L::kStages; ++s) { mbar_init(bar(BKF + s), 1); mbar_init(bar(BKE + s), 1); }
        mbar_fence_init();
        *s_abort = 0;
    }
    if (warp == 16) { tmem_alloc(smem_u32(s_tmem), 512); tmem_relinquish(); }
    if (warp == 17 && lane == 0) { tma_prefetch_desc(&mq); tma_prefetch_desc(&mk); tma_prefetch_desc(&mv); }
    // tables: the 32-way replicated fast-path table (one global load per entry, copies written
    // with 16-byte stores) and the plain full table
    {
        float4 *rep = reinterpret_cast<float4 *>(smem + L::kLutRepOff);
        for (int e = tid; e < kLutRepEntries; e += kTcThreads) {
            const float w = (e < 16) ? 1.f : g_w0_table[e - 16];
            const float4 w4 = make_float4(w, w, w, w);
#pragma unroll
            for (int i = 0; i < 8; ++i) rep[e * 8 + i] = w4;
        }
        float *full = reinterpret_cast<float *>(smem + L::kLutFullOff);
        for (int i = tid; i < kLutN; i += kTcThreads) full[i] = g_w0_table[i];
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *s_tmem;

    // Register budget: the fifth warpgroup (producer, MMA issuer, two idle warps) needs few
    // registers and hands part of its share to the sixteen softmax warps.  The pool is what the
    // CTA got at launch (640 x 96): 128 x 64 + 512 x 104 = 61440 uses it exactly; asking for more
    // than the pool holds would block forever.
    if (warp >= kTcSoftmaxWarps) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
      if (warp == 16) {
        // ======================= TMA producer ==================================================
        if (lane == 0) {
            const int nvalid = (jm[0] > 0) + (jm[1] > 0);
            mbar_arrive_expect_tx(bar(BQ), (uint32_t)(nvalid * L::kTileBytes));
            for (int t = 0; t < 2; ++t)
                if (jm[t] > 0)
                    for (int hh = 0; hh < D / 64; ++hh)
                        tma_load_2d(sbase + L::kQOff + t * L::kTileBytes + hh * 16384, &mq, hh * 64,
                                    q_row0 + t * 128, bar(BQ));
            int issued = 0;
            for (int l = 0; l < 2 * J; ++l) {
                const int s = l % L::kStages, n = l / L::kStages;
                if (n > 0 && !mbar_wait(bar(BKE + s), (uint32_t)((n - 1) & 1), s_abort, &g_async_status, 0x100 + s))
                    break;
                mbar_arrive_expect_tx(bar(BKF + s), (uint32_t)L::kTileBytes);
                const CUtensorMap *m = (l & 1) ? &mv : &mk;
                for (int hh = 0; hh < D / 64; ++hh)
                    tma_load_2d(sbase + L::kKvOff + s * L::kTileBytes + hh * 16384, m, hh * 64,
                                kv_row0 + (l >> 1) * 128, bar(BKF + s));
                issued = l + 1;
            }
            if (*s_abort) {
                // let copies already in flight land before the CTA's shared memory is released
                const int first = issued > L::kStages ? issued - L::kStages : 0;
                for (int l = first; l < issued; ++l) {
                    const int s = l % L::kStages, n = l / L::kStages;
                    const uint64_t t0 = globaltimer_ns();
                    while (!mbar_try_wait(bar(BKF + s), (uint32_t)(n & 1)) && globaltimer_ns() - t0 < 2000000ull) {}
                }
            }
        }
      } else if (warp == 17) {
        // ======================= MMA issuer ====================================================
        if (lane == 0) {
            constexpr uint32_t idesc_qk = make_idesc_bf16(128, 128, false);
            constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, true);
            const uint32_t o_cols = D;
            bool ok = mbar_wait(bar(BQ), 0, s_abort, &g_async_status, 0x200);
            auto kv_stage = [&](int l) { return l % L::kStages; };
            auto kv_parity = [&](int l) { return (uint32_t)((l / L::kStages) & 1); };
            auto issue_qk = [&](int t, int j) {
                const uint32_t qa = sbase + L::kQOff + t * L::kTileBytes;
                const uint32_t ka = sbase + L::kKvOff + kv_stage(2 * j) * L::kTileBytes;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = (uint32_t)((ks >> 2) * 16384 + (ks & 3) * 32);
                    mma_ss(tmem + t * 128, make_sdesc(qa + off, 16, 1024), make_sdesc(ka + off, 16, 1024),
                           idesc_qk, ks > 0);
                }
                mma_commit(bar(BS + t));
            };
            // P V in two parts: part 0 uses the first 32 keys of each key half (K-steps 0, 1, 4, 5), which
            // the softmax warps hand over while they still work on the rest; part 1 the other four.
            auto issue_pv = [&](int t, int j, int part) {
                const uint32_t va = sbase + L::kKvOff + kv_stage(2 * j + 1) * L::kTileBytes;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int ks = (i >> 1) * 4 + part * 2 + (i & 1);   // keys 16 ks ..
                    // P of key half h sits at columns 64 h .. of the tile's S region
                    mma_ts(tmem + 256 + t * o_cols, tmem + t * 128 + (ks >> 2) * 64 + (ks & 3) * 8,
                           make_sdesc(va + ks * 2048, 16384, 1024), idesc_pv, (j > 0 || part > 0 || i > 0) ? 1u : 0u);
                }
            };
            if (ok && J > 0) {
                ok = mbar_wait(bar(BKF + kv_stage(0)), kv_parity(0), s_abort, &g_async_status, 0x210);
                if (ok) {
                    tc_fence_after_sync();
                    for (int t = 0; t < 2; ++t)
                        if (jm[t] > 0) issue_qk(t, 0);
                    mma_commit(bar(BKE + kv_stage(0)));
                }
            }
            for (int j = 0; ok && j < J; ++j) {
                ok = mbar_wait(bar(BKF + kv_stage(2 * j + 1)), kv_parity(2 * j + 1), s_abort, &g_async_status, 0x220);
                if (!ok) break;
                bool next_ready = false;
                for (int t = 0; ok && t < 2; ++t) {
                    if (j < jm[t]) {
                        ok = mbar_wait(bar(BPA + t), (uint32_t)(j & 1), s_abort, &g_async_status, 0x260 + t);
                        if (!ok) break;
                        tc_fence_after_sync();
                        issue_pv(t, j, 0);
#ifndef BAPS_EXP_TENSORONLY
#ifdef BAPS_EXP_POLLMMA
                        ok = mbar_wait_poll<BAPS_EXP_POLLMMA>(bar(BP + t), (uint32_t)(j & 1), s_abort, &g_async_status, 0x230 + t);
#else
                        ok = mbar_wait(bar(BP + t), (uint32_t)(j & 1), s_abort, &g_async_status, 0x230 + t);
#endif
                        if (!ok) break;
#endif
                        tc_fence_after_sync();
                        issue_pv(t, j, 1);
                        if (j == jm[t] - 1) mma_commit(bar(BO + t));
                    }
                    if (j + 1 < jm[t]) {
                        if (!next_ready) {
                            ok = mbar_wait(bar(BKF + kv_stage(2 * j + 2)), kv_parity(2 * j + 2), s_abort,
                                           &g_async_status, 0x240);
                            if (!ok) break;
                            tc_fence_after_sync();
                            next_ready = true;
                        }
                        issue_qk(t, j + 1);
#ifdef BAPS_TRACE
                        if (blockIdx.x == 0 && j < 512) g_trace_mma[(t * 512 + j) * 2 + 1] = clock64();
#endif
                    }
                }
                if (!ok) break;
                mma_commit(bar(BKE + kv_stage(2 * j + 1)));
                if (next_ready) mma_commit(bar(BKE + kv_stage(2 * j + 2)));
            }
        }
      }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 104;");
        // ======================= softmax warps ==================================================
        const int t = warp >> 3;                 // query tile of the pair
        const int hf = (warp >> 2) & 1;          // key half: columns 64 hf .. 64 hf + 63 of the tile
        const int q4 = warp & 3;                 // TMEM lane quarter
        const int row = q4 * 32 + lane;
        const int qi = 2 * pair + t;
        const int jmax = jm[t];
        const uint32_t lane_sel = (uint32_t)(q4 * 32) << 16;
        const uint32_t s_addr = tmem + lane_sel + t * 128 + hf * 64;      // my 64 score columns
        const uint32_t o_addr = tmem + lane_sel + 256 + t * D + hf * (D / 2);
        const uint32_t lut_full = sbase + L::kLutFullOff;
        const uint32_t tb = sbase + L::kLutRepOff + (uint32_t)lane * 4u;
        volatile float *x_mine = s_xchg + (t * 128 + row) * 2 + hf;
        volatile float *x_other = s_xchg + (t * 128 + row) * 2 + (hf ^ 1);
        const uint32_t bx = bar(BX + t * 4 + q4);
        uint32_t xphase = 0;
        const float c = p.c;
        const bool exact = !kExp2 && p.mode == BAPS_MODE_EXACT;
        const bool count_restarts = p.restarts != nullptr && q4 == 0 && hf == 0;
        // m: running max of Algorithm 1 (integer valued; real valued in the exact mode).
        // m_ref: the max O~ and d are currently expressed against.  All rescale factors are exact
        // powers of two, so instead of multiplying O~ by 2^(m_old - m_new) whenever the max moves,
        // the tile's weights are multiplied by 2^(m~ - m_ref); O~ is touched only if that
        // exponent grows past 64 (or past 8 in the exact mode, whose factors are not exact).
        // Both threads of a row take identical decisions; each keeps the partial sum d of its half.
        float m = -INFINITY, m_ref = 0.f, d = 0.f;
        int n_restart = 0;
        bool ok = true;

        for (int j = 0; j < jmax; ++j) {
            ok = mbar_wait(bar(BS + t), (uint32_t)(j & 1), s_abort, &g_async_status, 0x300 + t);
            if (!ok) break;
            tc_fence_after_sync();
            const bool diag = p.causal && (j == qi);
            const int col_base = hf * 64;        // first key column of my half inside the tile
            // ---- pass 1: maximum of my half row, exchanged with the partner thread ---------------
            float mx;
            {
                uint32_t r[64];
                tmem_ld32(s_addr, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
                tmem_ld32(s_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&r[32]));
                tmem_wait_ld();
                if (diag) {
#pragma unroll
                    for (int i = 0; i < 64; ++i) r[i] = (col_base + i > row) ? 0xFF800000u : r[i];
                }
                const float g0 = max8(&r[0]), g1 = max8(&r[8]), g2 = max8(&r[16]), g3 = max8(&r[24]);
                const float g4 = max8(&r[32]), g5 = max8(&r[40]), g6 = max8(&r[48]), g7 = max8(&r[56]);
                const float hm = max3(max3(g0, g1, g2), max3(g3, g4, g5), fmaxf(g6, g7));
                *x_mine = hm;
                mbar_arrive(bx);
                ok = BAPS_WAIT_PAIR(bx, xphase, s_abort, &g_async_status, 0x340 + t);
                if (!ok) break;
                xphase ^= 1u;
                mx = fmaxf(hm, *x_other);
            }
            // ---- decisions (Algorithm 1: B0 branch / restart test / max update) -----------------
            const bool hp = !kExp2 && ((j == 0) || exact);
            // T of the row maximum, formed exactly like every element's T (one FMA)
            const float um = (hp || kExp2) ? -1.f : fmaf(mx, c, -m);
            const bool posf = um > 0.f;                       // the row has a positive T
            const bool any_posf = __any_sync(0xffffffffu, posf);
            float t8 = 0.f;
            bool any_over = false;
            if (any_posf) {
                t8 = posf ? hif8_round(um) : 0.f;             // 8-bit T of the row maximum
                any_over = __any_sync(0xffffffffu, t8 > (float)p.lambda);
            }
            int *flags = s_flags + (t * 2 + (j & 1)) * 4;
            if (hf == 0 && lane == 0) { flags[q4] = any_over ? 1 : 0; mbar_arrive(bar(BF + 2 * t + (j & 1))); }
            bool restart_tile = false;
            if (any_posf || (count_restarts && !hp)) {
                // the restart decision is tile-wide: wait for the verdicts of all four lane quarters
                ok = BAPS_WAIT_FLAG(bar(BF + 2 * t + (j & 1)), (uint32_t)((j >> 1) & 1), s_abort, &g_async_status, 0x310 + t);
                if (!ok) break;
                restart_tile = (flags[0] | flags[1] | flags[2] | flags[3]) != 0;
            }
            if (count_restarts && restart_tile) ++n_restart;
            float m_new, mref_w;                    // T of this tile is taken against mref_w
            if constexpr (kExp2) {
                // Eq. (2): real-valued running max.  The product was rounded: step the max up by one
                // unit in the last place if the row maximum's T would come out positive, so that every
                // T of the tile is <= 0.
                float smax = mx * c;
                if (fmaf(mx, c, -smax) > 0.f)
                    smax = __uint_as_float(__float_as_uint(smax) + (smax >= 0.f ? 1u : 0xFFFFFFFFu));
                m_new = fmaxf(m, smax);
                mref_w = m_new;
                if (j > 0) {
                    // rescale factor 2^(m_old - m_new), 8-bit in and out (not a power of two): O~ and d
                    // are multiplied for real.  P V of the previous key tile has completed (its commit
                    // precedes the one that released this tile's scores) and the next one waits for P.
                    const float alpha = lds_f32(lut_full + 4u * (uint32_t)w0_index(m - m_new));
                    if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll 1
                        for (int ch = 0; ch < D / 32; ++ch) {
                            uint32_t o[16];
                            tmem_ld16(o_addr + ch * 16, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                            tmem_st16(o_addr + ch * 16, o);
                        }
                    }
                    d *= alpha;
                }
                m_ref = m_new;
            } else if (hp || restart_tile) {
                float smax = mx * c;
                if (!exact) {
                    smax = ceilf(smax);
                    // the product was rounded: make sure no T against the new max is positive
                    if (fmaf(mx, c, -smax) > 0.f) smax += 1.f;
                }
                m_new = fmaxf(m, smax);
                if (j == 0) m_ref = m_new;
                mref_w = hp ? m_ref : m_new;
            } else {
                m_new = m + fmaxf(0.f, ceilf(t8));  // delta = max(0, ceil(rowmax T8))
                mref_w = m;                          // weights 2^T8 * 2^-delta = 2^T8 against the old max
            }
            // ---- rebase O~ and d (rare): only when the exponent against m_ref grows too large -------
            {
                const float target = hp ? m_new : mref_w;
                const float kk = target - m_ref;
                const bool need = !kExp2 && (j > 0) && (kk > (exact ? 8.f : 64.f));
                if (__any_sync(0xffffffffu, need)) {
                    const float f = exact ? ex2_approx(-kk) : pow2_int(-kk);
#pragma unroll 1
                    for (int ch = 0; ch < D / 32; ++ch) {
                        uint32_t o[16];
                        tmem_ld16(o_addr + ch * 16, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
                        tmem_st16(o_addr + ch * 16, o);
                    }
                    d *= f;
                    m_ref = target;
                    if (hp) mref_w = m_ref;
                }
            }
            // weights are expressed against m_ref: factor 2^e, e = mref_w - m_ref in [0, 64]
            const float e_f = (hp || kExp2) ? 0.f : (mref_w - m_ref);
            const uint32_t escale = (uint32_t)(int)e_f * 0x00800080u;
            const float scale = pow2_int(e_f);
            // some row of this warp has T > 0 in a tile that was not restarted: the 8-column groups
            // holding those few entries are redone with the full table after the fast path
            const bool pos_tile = !hp && !restart_tile && any_posf;      // warp-uniform
            // ---- pass 2: weights -> bf16 P over score columns already read; row sum ----------------
            float sum = 0.f;
            {
                const float mnv = kExp2 ? -mref_w : mref_w * 7.52316384526264e-37f;    // 2^-120
                const float cnv = kExp2 ? c : -c * 7.52316384526264e-37f;
                const uint64_t cn2 = pack2(cnv, cnv), mn2 = pack2(mnv, mnv);
                uint64_t s01 = 0ull, s23 = 0ull;
#pragma unroll 1
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t r[16], pk[8];
                    tmem_ld16(s_addr + ch * 16, r);
                    tmem_wait_ld();
                    if (diag) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) r[i] = (col_base + ch * 16 + i > row) ? 0xFF800000u : r[i];
                    }
                    if (hp) {
                        sum += hp16(r, pk, c, mref_w);
                    } else {
                        fast16<kExp2>(r, pk, cn2, mn2, escale, tb, s01, s23);
                        if (pos_tile) {
#pragma unroll
                            for (int gg = 0; gg < 2; ++gg) {
                                const bool gpos = fmaf(max8(&r[gg * 8]), c, -mref_w) > 0.f;
                                if (__any_sync(0xffffffffu, gpos))
                                    sum += fix8(&r[gg * 8], &pk[gg * 4], c, mref_w, escale, lut_full);
                            }
                        }
                    }
                    // 16 scores (columns 16 ch ..) become 8 packed columns 8 ch .., all of them read before
                    tmem_st8(s_addr + ch * 8, pk);
                    if (ch == 1) {
                        // first 32 keys of my half are in place: the tensor core may start on them
                        tmem_wait_st();
                        tc_fence_before_sync();
                        mbar_arrive(bar(BPA + t));
                    }
                }
                float a0, a1, a2, a3;
                unpack2(s01, a0, a1); unpack2(s23, a2, a3);
                sum += (a0 + a1) + (a2 + a3);
            }
            d += sum * scale;
            m = m_new;
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(bar(BP + t));
        }

        // ---- epilogue: O = O~ / d (each thread: its half of the output columns) ---------------------
        if (ok && jmax > 0) ok = mbar_wait(bar(BO + t), 0, s_abort, &g_async_status, 0x320 + t);
        if (ok && jmax > 0) {
            // total denominator of the row = my half + the partner's
            *x_mine = d;
            mbar_arrive(bx);
            ok = mbar_wait_poll<0>(bx, xphase, s_abort, &g_async_status, 0x350 + t);
        }
        if (ok && jmax > 0) {
            tc_fence_after_sync();
            const float dtot = d + *x_other;
            const float dinv = 1.f / dtot;
            const size_t grow = (size_t)q_row0 + (size_t)t * 128 + row;   // row in [B*H*S]
            const int ocol0 = hf * (D / 2);
#pragma unroll 1
            for (int ch = 0; ch < D / 32; ++ch) {
                uint32_t r[16];
                tmem_ld16(o_addr + ch * 16, r);
                tmem_wait_ld();
                float o[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) o[i] = __uint_as_float(r[i]) * dinv;
                if (p.out) {
                    uint4 *dst = reinterpret_cast<uint4 *>(p.out + grow * D + ocol0 + ch * 16);
#pragma unroll
                    for (int i = 0; i < 2; ++i)
                        dst[i] = make_uint4(pack_bf16x2(o[8 * i], o[8 * i + 1]), pack_bf16x2(o[8 * i + 2], o[8 * i + 3]),
                                            pack_bf16x2(o[8 * i + 4], o[8 * i + 5]), pack_bf16x2(o[8 * i + 6], o[8 * i + 7]));
                }
                if (p.out_f32) {
                    float4 *dst = reinterpret_cast<float4 *>(p.out_f32 + grow * D + ocol0 + ch * 16);
#pragma unroll
                    for (int i = 0; i < 4; ++i) dst[i] = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
                }
            }
            if (hf == 0) {
                if (p.row_m) p.row_m[grow] = m;
                // d is held against m_ref; report it against the final max
                if (p.row_d) p.row_d[grow] = dtot * (exact ? ex2_approx(m_ref - m) : pow2_int(m_ref - m));
            }
            if (count_restarts && lane == 0)
                p.restarts[(size_t)(b * p.H + h) * p.nq + qi] = n_restart;
        }
    }

    // ---- teardown ---------------------------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 16) { __syncwarp(); tmem_dealloc(tmem, 512); }
}

// Host side: tensor maps, one-time table initialisation, launch.
inline baps_status attention_tc_launch(const void *q, const void *k, const void *v, void *out, int B, int H,
                                       int Hkv, int S, int D, int causal, int lambda, int mode, float c,
                                       const baps_stats &st, int /*num_sms*/, cudaStream_t stream)
{
    static bool table_ready[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BAPS_ERR_CUDA;
    {
    std::lock_guard<std::mutex> setup_lock(g_setup_mutex);
    if (!table_ready[dev]) {
        // first call on this device: fill the w0 table and wait for it (later calls may come on
        // any stream)
        w0_table_init_kernel<<<1, 320, 0, stream>>>();
        if (cudaGetLastError() != cudaSuccess) return BAPS_ERR_CUDA;
        ++g_launches;
        if (cudaStreamSynchronize(stream) != cudaSuccess) return BAPS_ERR_CUDA;
        table_ready[dev] = true;
    }
    }
    CUtensorMap mq, mk, mv;
    if (!make_tmap_bf16_rows(&mq, q, (uint64_t)B * H * S, (uint64_t)D, 128) ||
        !make_tmap_bf16_rows(&mk, k, (uint64_t)B * Hkv * S, (uint64_t)D, 128) ||
        !make_tmap_bf16_rows(&mv, v, (uint64_t)B * Hkv * S, (uint64_t)D, 128))
        return BAPS_ERR_CUDA;
    AttnTcParams p;
    p.out = reinterpret_cast<__nv_bfloat16 *>(out);
    p.out_f32 = st.out_f32; p.row_m = st.row_m; p.row_d = st.row_d; p.restarts = st.restarts;
    p.B = B; p.H = H; p.Hkv = Hkv; p.S = S; p.causal = causal; p.lambda = lambda; p.mode = mode; p.c = c;
    p.nq = S / 128; p.npairs = (p.nq + 1) / 2;
    const long long nblocks = (long long)p.npairs * B * H;
    if (nblocks > 0x7fffffffLL) return BAPS_ERR_UNSUPPORTED;
    auto launch = [&](auto kernel, int sm) -> baps_status {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, sm) != cudaSuccess)
            return BAPS_ERR_CUDA;
        kernel<<<(unsigned)nblocks, kTcThreads, sm, stream>>>(mq, mk, mv, p);
        return launch_status();
    };
    const bool exp2m = mode == BAPS_MODE_EXP2_HIF8;
    if (D == 128)
        return exp2m ? launch(attention_tc_kernel<128, true>, TcLayout<128>::kDynBytes)
                     : launch(attention_tc_kernel<128, false>, TcLayout<128>::kDynBytes);
    return exp2m ? launch(attention_tc_kernel<64, true>, TcLayout<64>::kDynBytes)
                 : launch(attention_tc_kernel<64, false>, TcLayout<64>::kDynBytes);
}

} // namespace baps
