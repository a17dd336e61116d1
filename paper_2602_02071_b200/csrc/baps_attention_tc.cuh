// Fused BAPS attention forward on the 5th-generation tensor cores (tcgen05, sm_100a).
//
// One CTA owns two consecutive 128-row query tiles (t = 0, 1) of one (batch, head) and walks the
// key tiles j in increasing order (Algorithm 1: tile 0 is the high-precision set B0, all later
// tiles are 8-bit tiles).  The unit of work is a task (t, j): S = Q_t K_j^T, softmax bookkeeping
// and weights P, O_t += P V_j.  Tasks run in the order (0,0) (1,0) (0,1) (1,1) ...; task k uses
// score buffer k % 2 of tensor memory, so the tensor core forms the scores of task k + 1 while
// the softmax warps work on task k, and no softmax warp ever waits for a product of its own
// previous task.  Roles, by warp (640 threads):
//   warps 0-15  softmax warps, all sixteen on the current task.  Warp w owns rows 32*(w%4) .. +31
//               (its TMEM lanes) and the 32 key columns of quarter w/4, i.e. a row is shared by
//               four threads.  Per task: read the 32 scores once into registers, quarter-row
//               maximum, exchange through shared memory; one reducing hardware barrier of the
//               sixteen warps orders the exchange and carries the tile-wide restart vote (B0 and
//               non-8-bit tiles: a plain barrier of the four warps of a lane quarter); decide
//               (B0 / restart / plain), form the weights
//               w = HiF8(2^HiF8(S*c - m~)) * 2^-delta through a bank-replicated table indexed by
//               the top bits of the fp32 pattern, and write them to TMEM as bf16 (exactly
//               representable) over score columns the thread itself has read.
//   warp 16     TMA producer: Q tiles once, then K_0, V_0, K_1, V_1, ... through a ring.
//   warp 17     MMA issuer: S = Q_t K_j^T (operands in shared memory, 128-byte swizzle) and
//               O_t += P V_j (P from TMEM, V as an MN-major shared operand), in bursts
//               PV(k), QK(k+2).  (Warps 18-19 idle: the fifth warpgroup exists so that its
//               registers can be handed to the softmax warps.)
// TMEM (512 columns): S buffer 0 | S buffer 1 | O_0 | O_1, 128 columns each (64 for O when
// D = 64).  The bf16 weights of column quarter q overwrite columns [32q, 32q + 16) of the buffer.
// Every wait on an mbarrier is bounded; on expiry the CTA raises an abort flag and records a code
// in the library's status word.  Every later wait then returns at once; the softmax warps still run
// through their task list so that the hardware barriers they share stay matched, and all roles
// meet at the common teardown.
#pragma once
#include <cuda_bf16.h>
#include "baps_common.cuh"
#include "baps_hif8.cuh"
#include "baps_sm100.cuh"
#include "baps_tables.cuh"
#include "baps_tma_host.cuh"

namespace baps {

#ifdef BAPS_TEST_SKIP_LOAD
// Test build only (never defined for the product library): index of the K / V tile load that the
// TMA producer leaves out, so that the role waiting for that tile runs into its time limit.  -1: none.
__device__ int g_test_skip_load = -1;
#endif

struct AttnTcParams {
    __nv_bfloat16 *out;       // [B,H,S,D] or null
    float *out_f32;           // optional
    float *row_m, *row_d;     // optional [B,H,S]
    int32_t *restarts;        // optional [B,H,S/128]
    int B, H, Hkv, S, causal, lambda, mode;
    int b0_last;              // B0 = {first, last visible key tile}; one query tile per CTA
    const float *q_scale;     // 8-bit Q / K only: per query tile [B,H,S/128] and per key tile [B,Hkv,S/128]
    const float *k_scale;     // dequantisation scales (powers of two); null otherwise
    float c;                  // log2(e) * scale
    int nq, npairs;           // query tiles; work items per head (pairs of query tiles, or single tiles)
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
    // barriers: q_full, s_full[2], p_full[2], pv_done[2], kv_full[stages], kv_empty[stages]
    static constexpr int kNumBars = 1 + 2 + 2 + 2 + 2 * kStages;
    static constexpr int kXchgOff = (kBarOff + kNumBars * 8 + 15) & ~15;   // float xchg[2][128][4]
    static constexpr int kMiscOff = kXchgOff + 2 * 128 * 4 * 4;            // tmem base, abort
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
// Hardware (named) barriers among the softmax warps: id 0 is __syncthreads.
__device__ __forceinline__ void named_bar_sync(uint32_t id, uint32_t nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
// Barrier that also ORs a predicate over all participating threads.
__device__ __forceinline__ bool named_bar_or(uint32_t id, uint32_t nthreads, bool pred)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, %2, %3, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)pred), "r"(id), "r"(nthreads)
        : "memory");
    return r != 0;
}
__device__ __forceinline__ float4 lds_f32x4(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts_u32x4(uint32_t addr, uint4 v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint4 lds_u32x4(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts_f32(uint32_t addr, float v)
{
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
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
__device__ __forceinline__ void fast16(const uint32_t *r, uint32_t *pk, uint64_t cn2, uint64_t mn2,
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

// Eight columns of a group that holds a positive T (rows whose maximum rose above the running max
// in a tile that was not restarted have a few of those; the fast path gave them weight 0).  Only
// the positive entries are touched: each is looked up in the positive window of the full table
// (0 < T < 4 because the tile passed the restart test), patched into its half of the packed
// register and returned as the amount to add to the row sum.  Lanes without a positive entry skip the
// patch (a plain divergent branch: a warp-wide vote per entry cost more than it saved); the caller
// reconverges the warp afterwards.
__device__ __forceinline__ float fix8(const uint32_t *x, uint32_t *pk4, float c, float mref, uint32_t escale,
                                      uint32_t lut_full)
{
    const uint32_t lut_pos = lut_full + 4u * (uint32_t)(kLutNegN - kLutPosLo);
    float add = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float u = fmaf(__uint_as_float(x[i]), c, -mref);
        if (u > 0.f) {                         // few lanes, if any: the others skip
            const uint32_t key = min(max(__float_as_uint(u) >> 19, (uint32_t)kLutPosLo), (uint32_t)kLutPosHi);
            const float w = lds_f32(lut_pos + 4u * key);
            add += w;
            const uint32_t half = (__float_as_uint(w) >> 16) + (escale & 0xFFFFu);   // exact in bf16
            pk4[i >> 1] = (i & 1) ? __byte_perm(pk4[i >> 1], half, 0x5410) : __byte_perm(pk4[i >> 1], half, 0x3254);
        }
    }
    return add;
}

// High-precision tile (B0, or every tile in the exact mode): P = 2^(S*c - mref) in fp32, rounded
// to bf16 for the tensor core; the row sum uses the rounded values so that numerator and
// denominator see the same weights.  Masked entries arrive as -inf and give 0.
__device__ __forceinline__ float hp16(const uint32_t *r, uint32_t *pk, float c, float mref)
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

// kQK8: Q and K arrive as E4M3 codes with one power-of-two scale per 128-row tile (the dequantisation
// the paper proposes to fuse, Section 3.4): Q K^T runs on the 8-bit tensor-core path and the two
// scales of a tile pair are folded into the score scale c, task by task.  D = 128 only.
// kB0Last: B0 = {first, last visible key tile} (compile-time, so that the usual order pays nothing).
// kMode (BAPS_MODE_*): Algorithm 1, the exact mode, or -- kExp2 below -- the "Exp2 HiF8" setup of Section 4.1 (Eq. (2) with a real-valued max, weights and
// rescale factor through the 8-bit exponent table); otherwise Algorithm 1 or the exact mode.
template <int D, int kMode, bool kQK8 = false, bool kB0Last = false>
__global__ void __launch_bounds__(kTcThreads, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mk,
                    const __grid_constant__ CUtensorMap mv, const AttnTcParams p)
{
    using namespace sm100;
    using L = TcLayout<D>;
    constexpr bool kExp2 = kMode == BAPS_MODE_EXP2_HIF8;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + L::kBarOff;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    // q_full | s_full[buffer] | p_full[buffer] | pv_done[query tile] | kv_full[stage] | kv_empty[stage]
    constexpr int BQ = 0, BS = 1, BP = 3, BD = 5, BKF = 7, BKE = 7 + L::kStages;
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
    // With B0 = {first, last} the key tiles are visited in the order 0, last, 1, ..., last - 1, and
    // "last" differs between neighbouring query tiles of a causal problem, so the two query tiles of
    // a pair could not share their K / V stream: the CTA then owns a single query tile (t = 0).
    const int qbase = kB0Last ? pair : 2 * pair;        // first query tile of this CTA
    int jm[2];                                   // number of key tiles of each query tile
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int qi = qbase + t;
        jm[t] = (qi < p.nq && !(kB0Last && t == 1)) ? (p.causal ? qi + 1 : nk) : 0;
    }
    const int J = jm[0] > jm[1] ? jm[0] : jm[1];
    const int nb0 = (kB0Last && J >= 2) ? 2 : 1;        // number of high-precision (B0) steps
    // key tile visited at step s
    auto key_tile = [&](int s) { return !kB0Last ? s : (s == 0 ? 0 : (s == 1 ? J - 1 : s - 1)); };
    const int q_row0 = (b * p.H + h) * p.S + qbase * 128;           // row in the [B*H*S, D] view
    const int kv_row0 = (b * p.Hkv + hk) * p.S;

    // ---- setup --------------------------------------------------------------------------------
    // kEarly (D = 64, where a CTA lives for few tasks): the producer lane initialises the barriers itself and
    // starts the Q tiles and the first ring-full of K / V tiles before the CTA-wide barrier, so that the copies
    // are on their way while the rest of the CTA is still setting up.  (At D = 128 the same change made the
    // steady state 2 % slower, so that path keeps the plain order.)
    constexpr bool kEarly = (D == 64);
    constexpr int kQkBoxes = kQK8 ? 1 : D / 64;
    constexpr uint32_t kQkTileBytes = kQK8 ? 128 * D : L::kTileBytes;
    const int n_early = kEarly ? (2 * J < L::kStages ? 2 * J : L::kStages) : 0;   // loads that need no free stage
    if constexpr (kEarly) {
        if (tid == 0) *s_abort = 0;
        if (warp == 16) {
            if (lane == 0) {
                mbar_init(bar(BQ), 1);
                for (int i = 0; i < 2; ++i) {
                    mbar_init(bar(BS + i), 1);
                    mbar_init(bar(BP + i), kTcSoftmaxWarps * 32);
                    mbar_init(bar(BD + i), 1);
                }
                for (int s = 0; s < L::kStages; ++s) { mbar_init(bar(BKF + s), 1); mbar_init(bar(BKE + s), 1); }
                mbar_fence_init();
                const int nvalid = (jm[0] > 0) + (jm[1] > 0);
                mbar_arrive_expect_tx(bar(BQ), (uint32_t)nvalid * kQkTileBytes);
                for (int t = 0; t < 2; ++t)
                    if (jm[t] > 0)
                        for (int hh = 0; hh < kQkBoxes; ++hh)
                            tma_load_2d(sbase + L::kQOff + t * L::kTileBytes + hh * 16384, &mq, hh * 64,
                                        q_row0 + t * 128, bar(BQ));
                for (int l = 0; l < n_early; ++l) {
#ifdef BAPS_TEST_SKIP_LOAD
                    if (l == g_test_skip_load) continue;      // this tile never arrives
#endif
                    const int s = l % L::kStages;
                    mbar_arrive_expect_tx(bar(BKF + s), (l & 1) ? (uint32_t)L::kTileBytes : kQkTileBytes);
                    const CUtensorMap *m = (l & 1) ? &mv : &mk;
                    for (int hh = 0; hh < ((l & 1) ? D / 64 : kQkBoxes); ++hh)
                        tma_load_2d(sbase + L::kKvOff + s * L::kTileBytes + hh * 16384, m, hh * 64,
                                    kv_row0 + key_tile(l >> 1) * 128, bar(BKF + s));
                }
            }
            __syncwarp();
            tmem_alloc(smem_u32(s_tmem), 512); tmem_relinquish();
        }
    } else {
        if (tid == 0) {
            mbar_init(bar(BQ), 1);
            for (int i = 0; i < 2; ++i) {
                mbar_init(bar(BS + i), 1);
                mbar_init(bar(BP + i), kTcSoftmaxWarps * 32);
                mbar_init(bar(BD + i), 1);
            }
            for (int s = 0; s < L::kStages; ++s) { mbar_init(bar(BKF + s), 1); mbar_init(bar(BKE + s), 1); }
            mbar_fence_init();
            *s_abort = 0;
        }
        if (warp == 16) { tmem_alloc(smem_u32(s_tmem), 512); tmem_relinquish(); }
    }
    if (warp == 17 && lane == 0) { tma_prefetch_desc(&mq); tma_prefetch_desc(&mk); tma_prefetch_desc(&mv); }
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
            if constexpr (!kEarly) {
                const int nvalid = (jm[0] > 0) + (jm[1] > 0);
                mbar_arrive_expect_tx(bar(BQ), (uint32_t)nvalid * kQkTileBytes);
                for (int t = 0; t < 2; ++t)
                    if (jm[t] > 0)
                        for (int hh = 0; hh < kQkBoxes; ++hh)
                            tma_load_2d(sbase + L::kQOff + t * L::kTileBytes + hh * 16384, &mq, hh * 64,
                                        q_row0 + t * 128, bar(BQ));
            }
            int issued = n_early;
            for (int l = n_early; l < 2 * J; ++l) {
                const int s = l % L::kStages, n = l / L::kStages;
                if (n > 0 && !mbar_wait(bar(BKE + s), (uint32_t)((n - 1) & 1), s_abort, &g_async_status, 0x100 + s))
                    break;
#ifdef BAPS_TEST_SKIP_LOAD
                if (l == g_test_skip_load) continue;          // this tile never arrives
#endif
                mbar_arrive_expect_tx(bar(BKF + s), (l & 1) ? (uint32_t)L::kTileBytes : kQkTileBytes);
                const CUtensorMap *m = (l & 1) ? &mv : &mk;
                for (int hh = 0; hh < ((l & 1) ? D / 64 : kQkBoxes); ++hh)
                    tma_load_2d(sbase + L::kKvOff + s * L::kTileBytes + hh * 16384, m, hh * 64,
                                kv_row0 + key_tile(l >> 1) * 128, bar(BKF + s));
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
        // The whole warp runs the loop (waits, task bookkeeping, descriptor arithmetic) so that the
        // compiler can keep it on the uniform datapath; one elected lane issues the MMAs and commits.
        {
            constexpr uint32_t idesc_qk = make_idesc_bf16(128, 128, false);
            constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, true);
            auto kv_stage = [&](int l) { return l % L::kStages; };
            auto kv_parity = [&](int l) { return (uint32_t)((l / L::kStages) & 1); };
            // the last query tile that uses key tile j: its MMA releases the K / V stage
            auto last_user = [&](int j) { return (j < jm[1]) ? 1 : 0; };
            // task order (0,0) (1,0) (0,1) (1,1) ... restricted to j < jm[t]
            auto advance = [&](int &t, int &j) -> bool {
                if (t == 0 && j < jm[1]) { t = 1; return true; }
                ++j;
                if (j < jm[0]) { t = 0; return true; }
                if (j < jm[1]) { t = 1; return true; }
                return false;
            };
            auto wait_all = [&](uint32_t bar_addr, uint32_t parity, int code) -> bool {
                return __all_sync(0xffffffffu, mbar_wait(bar_addr, parity, s_abort, &g_async_status, code));
            };
            bool ok = wait_all(bar(BQ), 0, 0x200);
            int k_ready = -1, v_ready = -1;      // key / value tiles whose arrival has been awaited
            auto await_k = [&](int j) -> bool {
                if (j <= k_ready) return true;
                if (!wait_all(bar(BKF + kv_stage(2 * j)), kv_parity(2 * j), 0x210)) return false;
                k_ready = j;
                return true;
            };
            auto await_v = [&](int j) -> bool {
                if (j <= v_ready) return true;
                if (!wait_all(bar(BKF + kv_stage(2 * j + 1)), kv_parity(2 * j + 1), 0x220)) return false;
                v_ready = j;
                return true;
            };
            // S buffer (k & 1) = Q_t K_j^T (issuing lane only)
            auto mma_qk = [&](int t, int j, int k) {
                const uint32_t qd = sdesc_lo(sbase + L::kQOff + t * L::kTileBytes, 16);
                const uint32_t kd = sdesc_lo(sbase + L::kKvOff + kv_stage(2 * j) * L::kTileBytes, 16);
                const uint32_t sd = tmem + (k & 1) * 128;
                if constexpr (kQK8) {
                    // rows of 128 E4M3 bytes: K = 32 per instruction, 32 bytes further along the row each
                    constexpr uint32_t idesc_qk8 = make_idesc_e4m3(128, 128);
#pragma unroll
                    for (int ks = 0; ks < D / 32; ++ks)
                        mma_ss_lo_f8(sd, qd + 2u * ks, kd + 2u * ks, idesc_qk8, ks > 0);
                } else {
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        const uint32_t off = (uint32_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4);
                        mma_ss_lo(sd, qd + off, kd + off, idesc_qk, ks > 0);
                    }
                }
                mma_commit(bar(BS + (k & 1)));
            };
            // O_t += P V_j with P in S buffer (k & 1): the weights of keys 16 ks .. 16 ks + 15 sit at
            // columns 32 (ks / 2) + 8 (ks % 2) of the buffer (issuing lane only)
            auto mma_pv = [&](int t, int j, int k) {
                const uint32_t vd = sdesc_lo(sbase + L::kKvOff + kv_stage(2 * j + 1) * L::kTileBytes, 16384);
                const uint32_t od = tmem + 256 + t * D, pd = tmem + (k & 1) * 128;
                const uint32_t acc0 = j > 0 ? 1u : 0u;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    mma_ts_lo(od, pd + (ks >> 1) * 32 + (ks & 1) * 8, vd + ks * 128, idesc_pv, ks > 0 ? 1u : acc0);
            };
            const bool leader = elect_one();
            if (ok && J > 0) {
                int t = 0, j = 0, k = 0;          // task whose P V comes next
                int tq = 0, jq = 0, kq = 0;       // task whose Q K^T comes next
                bool more_q = true;
                // scores of the first two tasks: both buffers are free
                for (int i = 0; i < 2 && ok && more_q; ++i) {
                    ok = await_k(jq);
                    if (!ok) break;
                    tc_fence_after_sync();
                    if (leader) {
                        mma_qk(tq, jq, kq);
                        if (tq == last_user(jq)) mma_commit(bar(BKE + kv_stage(2 * jq)));
                    }
                    __syncwarp();
                    more_q = advance(tq, jq);
                    ++kq;
                }
                while (ok) {
                    // One burst per task: P V of task k, then at once Q K^T of task k + 2 into the buffer
                    // P V reads (the tensor core runs them in order), so that the softmax warps find the
                    // scores of task k + 2 ready when they get there.  Everything the burst needs except P
                    // is awaited before P.
                    ok = await_v(j);
                    if (ok && more_q) ok = await_k(jq);
                    if (!ok) break;
                    ok = wait_all(bar(BP + (k & 1)), (uint32_t)((k >> 1) & 1), 0x230 + (k & 1));
                    if (!ok) break;
                    tc_fence_after_sync();
                    if (leader) {
                        mma_pv(t, j, k);
                        if (more_q) mma_qk(tq, jq, kq);
                        mma_commit(bar(BD + t));
                        if (t == last_user(j)) mma_commit(bar(BKE + kv_stage(2 * j + 1)));
                        if (more_q && tq == last_user(jq)) mma_commit(bar(BKE + kv_stage(2 * jq)));
                    }
                    __syncwarp();
                    if (more_q) { more_q = advance(tq, jq); ++kq; }
                    if (!advance(t, j)) break;
                    ++k;
                }
            }
        }
      }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 104;");
        // ======================= softmax warps ==================================================
        // Tables, built while the first Q / K tiles are on their way: the 32-way replicated fast-path
        // table (one global load per entry, copies written with 16-byte stores) and the plain full
        // table.  Only the softmax warps read them, so a barrier among these warps suffices.
        {
            float4 *rep = reinterpret_cast<float4 *>(smem + L::kLutRepOff);
            for (int e = tid; e < kLutRepEntries; e += kTcSoftmaxWarps * 32) {
                const float w = (e < 16) ? 1.f : g_w0_table[e - 16];
                const float4 w4 = make_float4(w, w, w, w);
#pragma unroll
                for (int i = 0; i < 8; ++i) rep[e * 8 + i] = w4;
            }
            float *full = reinterpret_cast<float *>(smem + L::kLutFullOff);
            for (int i = tid; i < kLutN; i += kTcSoftmaxWarps * 32) full[i] = g_w0_table[i];
            named_bar_sync(6, kTcSoftmaxWarps * 32);
        }
        const int q4 = warp & 3;                 // TMEM lane quarter: rows 32 q4 .. 32 q4 + 31
        const int cq = warp >> 2;                // key column quarter: columns 32 cq .. 32 cq + 31
        const int row = q4 * 32 + lane;
        const uint32_t lane_sel = (uint32_t)(q4 * 32) << 16;
        const uint32_t s_col = tmem + lane_sel + cq * 32;                 // + 128 * buffer
        const uint32_t lut_full = sbase + L::kLutFullOff;
        const uint32_t tb = sbase + L::kLutRepOff + (uint32_t)lane * 4u;
        const uint32_t xrow = sbase + L::kXchgOff + (uint32_t)row * 16u;  // + 2048 * (k & 1); my slot + 4 cq
        const float c_base = p.c;
        constexpr bool exact = kMode == BAPS_MODE_EXACT;
        constexpr bool e2e = kMode == BAPS_MODE_E2E_HIF8;
        const bool count_restarts = p.restarts != nullptr && warp == 0;
        // HiF8(T) > lambda  <=>  T >= the midpoint between lambda and the next HiF8 value above it
        // (rounding is monotone, ties go up): 2^-23 | 1.0625 | 2.125 | 3.125 for lambda 0 | 1 | 2 | 3.
        const float over_thr = p.lambda == 0 ? 1.1920928955078125e-07f
                                             : (float)p.lambda + (p.lambda == 1 ? 0.0625f : 0.125f);
        // Per query tile t: m, the running max of Algorithm 1 (integer valued; real valued in the exact
        // and Exp2 modes); m_ref, the max O~ and d are currently expressed against.  All rescale
        // factors of Algorithm 1 are exact powers of two, so instead of multiplying O~ by
        // 2^(m_old - m_new) whenever the max moves, the tile's weights are multiplied by
        // 2^(m~ - m_ref); O~ is touched only if that exponent grows past 64 (or past 8 in the exact
        // mode, whose factors are not exact).  The four threads of a row take identical decisions; each
        // keeps the partial sum d of its column quarter.
        float m[2] = {-INFINITY, -INFINITY}, m_ref[2] = {0.f, 0.f}, d[2] = {0.f, 0.f};
        int n_restart[2] = {0, 0};
        int k = 0;                               // running task index
        uint32_t r[32];                          // scores of the current task (my quarter row)

        // One task.  T is a compile-time query tile so that the per-tile state stays in registers.
        // Scores of task k_ -> r (asynchronous; completed by tmem_wait_ld at the start of the task).
        auto load_scores = [&](int k_) {
            mbar_wait(bar(BS + (k_ & 1)), (uint32_t)((k_ >> 1) & 1), s_abort, &g_async_status, 0x300 + (k_ & 1));
            tc_fence_after_sync();
            tmem_ld32(s_col + (uint32_t)(k_ & 1) * 128u, r);
        };
        auto task = [&](auto tconst, const int j, const bool has_next) {
            constexpr int T = decltype(tconst)::value;
            const int qi = qbase + T;
            // score scale of this task: log2(e) * scale, times the dequantisation scales of the query tile
            // and of the key tile when Q and K are 8-bit (powers of two: the product is exact)
            float c = c_base;
            if constexpr (kQK8)
                c = c_base * __ldg(p.q_scale + (size_t)(b * p.H + h) * p.nq + qi) *
                    __ldg(p.k_scale + (size_t)(b * p.Hkv + hk) * nk + key_tile(j));
            const uint32_t s_addr = s_col + (uint32_t)(k & 1) * 128u;
            const uint32_t x_addr = xrow + (uint32_t)(k & 1) * 2048u;
            const bool diag = p.causal && (key_tile(j) == qi);
            // ---- scores of my quarter row, their maximum, exchange with the three partner threads ----
            tmem_wait_ld();
            if (diag) {
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = (cq * 32 + i > row) ? 0xFF800000u : r[i];
            }
            const bool hp = !kExp2 && ((j < nb0) || exact);
            const float g[4] = {max8(&r[0]), max8(&r[8]), max8(&r[16]), max8(&r[24])};
            float mx;
            bool restart_tile = false;
            {
                const float hm = fmaxf(fmaxf(g[0], g[1]), fmaxf(g[2], g[3]));
                sts_f32(x_addr + 4u * (uint32_t)cq, hm);
                if (e2e && j >= nb0) {
                    // The restart decision is tile-wide: does any row have HiF8(T of its maximum) >
                    // lambda?  The test is monotone, so a row passes it iff one of its quarters does:
                    // one reducing barrier over all softmax threads gives the verdict and also orders
                    // the exchange of the quarter maxima.
                    restart_tile = named_bar_or(5, kTcSoftmaxWarps * 32, fmaf(hm, c, -m[T]) >= over_thr);
                    if (count_restarts && restart_tile) ++n_restart[T];
                } else {
                    named_bar_sync(1 + q4, 128);
                }
                const float4 pm = lds_f32x4(x_addr);
                mx = fmaxf(fmaxf(pm.x, pm.y), fmaxf(pm.z, pm.w));
            }
            // ---- decisions (Algorithm 1: B0 branch / restart test / max update) -----------------
            // T of the row maximum, formed exactly like every element's T (one FMA)
            const float um = (hp || kExp2) ? -1.f : fmaf(mx, c, -m[T]);
            const bool posf = um > 0.f;                       // the row has a positive T
            const bool any_posf = __any_sync(0xffffffffu, posf);
            float m_new, mref_w;                    // T of this tile is taken against mref_w
            if constexpr (kExp2) {
                // Eq. (2): real-valued running max.  The product was rounded: step the max up by one
                // unit in the last place if the row maximum's T would come out positive, so that every
                // T of the tile is <= 0.
                float smax = mx * c;
                if (fmaf(mx, c, -smax) > 0.f)
                    smax = __uint_as_float(__float_as_uint(smax) + (smax >= 0.f ? 1u : 0xFFFFFFFFu));
                m_new = fmaxf(m[T], smax);
                mref_w = m_new;
                if (j > 0) {
                    // rescale factor 2^(m_old - m_new), 8-bit in and out (not a power of two): O~ and d
                    // are multiplied for real, once P V of this query tile's previous task is complete.
                    const float alpha = lds_f32(lut_full + 4u * (uint32_t)w0_index(m[T] - m_new));
                    if (__any_sync(0xffffffffu, alpha != 1.f)) {
                        mbar_wait(bar(BD + T), (uint32_t)((j - 1) & 1), s_abort, &g_async_status, 0x330 + T);
                        tc_fence_after_sync();
                        const uint32_t o_addr = tmem + lane_sel + 256 + T * D + cq * (D / 4);
#pragma unroll 1
                        for (int ch = 0; ch < D / 64; ++ch) {
                            uint32_t o[16];
                            tmem_ld16(o_addr + ch * 16, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                            tmem_st16(o_addr + ch * 16, o);
                        }
                    }
                    d[T] *= alpha;
                }
                m_ref[T] = m_new;
            } else if (hp || restart_tile) {
                float smax = mx * c;
                if (!exact) {
                    smax = ceilf(smax);
                    // the product was rounded: make sure no T against the new max is positive
                    if (fmaf(mx, c, -smax) > 0.f) smax += 1.f;
                }
                m_new = fmaxf(m[T], smax);
                if (j == 0) m_ref[T] = m_new;
                mref_w = hp ? m_ref[T] : m_new;
            } else {
                // delta = max(0, ceil(rowmax T8)); weights 2^T8 * 2^-delta = 2^T8 against the old max.
                // The tile passed the restart test, so T < 3.125, and ceil(HiF8(T)) only depends on which
                // rounding midpoints T has reached: 0 below 2^-23 (rounds to 0), else 1 below 1.0625,
                // else 2 below 2.125, else 3.
                const float delta = (um >= 1.1920928955078125e-07f ? 1.f : 0.f) + (um >= 1.0625f ? 1.f : 0.f) +
                                    (um >= 2.125f ? 1.f : 0.f);
                m_new = m[T] + delta;
                mref_w = m[T];
            }
            // ---- rebase O~ and d (rare): only when the exponent against m_ref grows too large -------
            if constexpr (!kExp2) {
                const float target = hp ? m_new : mref_w;
                const float kk = target - m_ref[T];
                const bool need = (j > 0) && (kk > (exact ? 8.f : 64.f));
                if (__any_sync(0xffffffffu, need)) {
                    const float f = need ? (exact ? ex2_approx(-kk) : pow2_int(-kk)) : 1.f;
                    mbar_wait(bar(BD + T), (uint32_t)((j - 1) & 1), s_abort, &g_async_status, 0x330 + T);
                    tc_fence_after_sync();
                    const uint32_t o_addr = tmem + lane_sel + 256 + T * D + cq * (D / 4);
#pragma unroll 1
                    for (int ch = 0; ch < D / 64; ++ch) {
                        uint32_t o[16];
                        tmem_ld16(o_addr + ch * 16, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
                        tmem_st16(o_addr + ch * 16, o);
                    }
                    d[T] *= f;
                    if (need) {
                        m_ref[T] = target;
                        if (hp) mref_w = target;
                    }
                }
            }
            // weights are expressed against m_ref: factor 2^e, e = mref_w - m_ref in [0, 64]
            const float e_f = (hp || kExp2) ? 0.f : (mref_w - m_ref[T]);
            const int e_i = (int)e_f;                 // 0 .. 64 (the rebase above keeps it there)
            const uint32_t escale = (uint32_t)e_i * 0x00800080u;
            // some row of this warp has T > 0 in a tile that was not restarted: the 8-column groups
            // holding those few entries are redone with the full table after the fast path
            const bool pos_tile = e2e && !hp && !restart_tile && any_posf;      // warp-uniform
            // ---- weights -> bf16 P over score columns already read; row sum ---------------------------
            float sum = 0.f;
            uint32_t pk[16];
            if (hp) {
                sum = hp16(&r[0], &pk[0], c, mref_w) + hp16(&r[16], &pk[8], c, mref_w);
            } else {
                // (8-bit Q / K: c carries the dequantisation scales and may be far too small for the
                // combined constant c * 2^-120 to be a normal number, hence the two-step form there too)
                constexpr bool kTwo = kExp2 || kQK8;
                const float mnv = kTwo ? -mref_w : mref_w * 7.52316384526264e-37f;    // 2^-120
                const float cnv = kTwo ? c : -c * 7.52316384526264e-37f;
                const uint64_t cn2 = pack2(cnv, cnv), mn2 = pack2(mnv, mnv);
                uint64_t s01 = 0ull, s23 = 0ull;
                fast16<kTwo>(&r[0], &pk[0], cn2, mn2, escale, tb, s01, s23);
                fast16<kTwo>(&r[16], &pk[8], cn2, mn2, escale, tb, s01, s23);
                if (pos_tile) {
#pragma unroll
                    for (int gg = 0; gg < 4; ++gg) {
                        const bool gpos = fmaf(g[gg], c, -mref_w) > 0.f;
                        if (__any_sync(0xffffffffu, gpos))
                            sum += fix8(&r[gg * 8], &pk[gg * 4], c, mref_w, escale, lut_full);
                        __syncwarp();
                    }
                }
                float a0, a1, a2, a3;
                unpack2(s01, a0, a1); unpack2(s23, a2, a3);
                sum += (a0 + a1) + (a2 + a3);
            }
            // 32 scores (columns 32 cq ..) become 16 packed columns 32 cq .. 32 cq + 15
            tmem_st16(s_addr, pk);
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(bar(BP + (k & 1)));       // P is in place: the tensor core's burst may go
            d[T] += sum * __int_as_float((127 + e_i) << 23);
            m[T] = m_new;
            // the next task's scores travel into registers while the loop turns around
            if (has_next) load_scores(k + 1);
            ++k;
        };

        if (J > 0) load_scores(0);
        for (int j = 0; j < J; ++j) {
            if (j < jm[0]) task(std::integral_constant<int, 0>{}, j, j < jm[1] || j + 1 < J);
            if (j < jm[1]) task(std::integral_constant<int, 1>{}, j, j + 1 < J);
        }
        const bool ok = (*s_abort == 0);

        // ---- epilogue: O = O~ / d (each thread: its quarter of the output columns) ---------------------
        auto finish = [&](auto tconst) {
            constexpr int T = decltype(tconst)::value;
            const int jmax = jm[T];
            if (jmax == 0) return;                                   // uniform over the CTA
            const int qi = qbase + T;
            const bool done = mbar_wait(bar(BD + T), (uint32_t)((jmax - 1) & 1), s_abort, &g_async_status, 0x320 + T);
            tc_fence_after_sync();
            // total denominator of the row = the four quarter sums
            // the exchange buffer not used by the task before (that one may still be read by a partner)
            const uint32_t x_addr = xrow + (uint32_t)((k + T) & 1) * 2048u;
            sts_f32(x_addr + 4u * (uint32_t)cq, d[T]);
            named_bar_sync(1 + q4, 128);
            const float4 pd = lds_f32x4(x_addr);
            const float dtot = (pd.x + pd.y) + (pd.z + pd.w);
            const bool good = ok && done;
            const float dinv = 1.f / dtot;
            const size_t grow = (size_t)q_row0 + (size_t)T * 128 + row;   // row in [B*H*S]
            const int ocol0 = cq * (D / 4);
            const uint32_t o_addr = tmem + lane_sel + 256 + T * D + ocol0;
            // The bf16 output goes through the (now idle) Q staging area of this tile so that the global
            // stores are whole rows: a thread owns 32 columns of one row, i.e. a warp's direct stores
            // would touch 32 rows with 16 bytes each.  Staged layout: row-major, the 16-byte chunks of a
            // row XOR-swizzled with the row number (conflict-free both ways).
            constexpr int kRowBytes = D * 2, kChunks = kRowBytes / 16;
            const uint32_t stage = sbase + L::kQOff + T * L::kTileBytes;
#pragma unroll 1
            for (int ch = 0; ch < D / 64; ++ch) {
                uint32_t rr[16];
                tmem_ld16(o_addr + ch * 16, rr);
                tmem_wait_ld();
                float o[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) o[i] = __uint_as_float(rr[i]) * dinv;
                if (p.out) {
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        const int chunk = (ocol0 + ch * 16) / 8 + i;
                        sts_u32x4(stage + (uint32_t)row * kRowBytes + (uint32_t)((chunk ^ (row & (kChunks - 1))) * 16),
                                  make_uint4(pack_bf16x2(o[8 * i], o[8 * i + 1]), pack_bf16x2(o[8 * i + 2], o[8 * i + 3]),
                                             pack_bf16x2(o[8 * i + 4], o[8 * i + 5]), pack_bf16x2(o[8 * i + 6], o[8 * i + 7])));
                    }
                }
                if (p.out_f32 && good) {
                    float4 *dst = reinterpret_cast<float4 *>(p.out_f32 + grow * D + ocol0 + ch * 16);
#pragma unroll
                    for (int i = 0; i < 4; ++i) dst[i] = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
                }
            }
            if (p.out) {
                // the four warps of a lane quarter staged the 32 rows of that quarter; each now writes eight
                // of them, 512 contiguous bytes per instruction
                named_bar_sync(1 + q4, 128);
                constexpr int kRowsPerInstr = 32 / kChunks;              // 2 (D = 128) or 4 (D = 64)
#pragma unroll
                for (int it = 0; it < 8 / kRowsPerInstr; ++it) {
                    const int rw = q4 * 32 + cq * 8 + it * kRowsPerInstr + lane / kChunks;
                    const int chunk = lane % kChunks;
                    const uint4 v = lds_u32x4(stage + (uint32_t)rw * kRowBytes + (uint32_t)((chunk ^ (rw & (kChunks - 1))) * 16));
                    if (good)
                        *reinterpret_cast<uint4 *>(reinterpret_cast<uint8_t *>(p.out) +
                                                   ((size_t)q_row0 + (size_t)T * 128 + rw) * kRowBytes + chunk * 16) = v;
                }
            }
            if (!good) return;
            if (cq == 0) {
                if (p.row_m) p.row_m[grow] = m[T];
                // d is held against m_ref; report it against the final max
                if (p.row_d) p.row_d[grow] = dtot * (exact ? ex2_approx(m_ref[T] - m[T]) : pow2_int(m_ref[T] - m[T]));
            }
            if (count_restarts && lane == 0)
                p.restarts[(size_t)(b * p.H + h) * p.nq + qi] = n_restart[T];
        };
        finish(std::integral_constant<int, 0>{});
        finish(std::integral_constant<int, 1>{});
    }

    // ---- teardown ---------------------------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 16) { __syncwarp(); tmem_dealloc(tmem, 512); }
}

// Host side: tensor maps, one-time table initialisation, launch.
static inline baps_status attention_tc_launch(const void *q, const void *k, const void *v, void *out, int B, int H,
                                       int Hkv, int S, int D, int causal, int lambda, int mode, int b0_last, float c,
                                       const baps_stats &st, int /*num_sms*/, cudaStream_t stream,
                                       const float *q_scale = nullptr, const float *k_scale = nullptr)
{
    const bool qk8 = q_scale != nullptr;               // Q, K are E4M3 codes with per-tile scales
    const baps_status ts = ensure_w0_table(stream);
    if (ts != BAPS_OK) return ts;
    CUtensorMap mq, mk, mv;
    if (qk8) {
        if (!make_tmap_u8_rows(&mq, q, (uint64_t)B * H * S, (uint64_t)D, 128) ||
            !make_tmap_u8_rows(&mk, k, (uint64_t)B * Hkv * S, (uint64_t)D, 128))
            return BAPS_ERR_CUDA;
    } else if (!make_tmap_bf16_rows(&mq, q, (uint64_t)B * H * S, (uint64_t)D, 128) ||
               !make_tmap_bf16_rows(&mk, k, (uint64_t)B * Hkv * S, (uint64_t)D, 128)) {
        return BAPS_ERR_CUDA;
    }
    if (!make_tmap_bf16_rows(&mv, v, (uint64_t)B * Hkv * S, (uint64_t)D, 128)) return BAPS_ERR_CUDA;
    AttnTcParams p;
    p.out = reinterpret_cast<__nv_bfloat16 *>(out);
    p.out_f32 = st.out_f32; p.row_m = st.row_m; p.row_d = st.row_d; p.restarts = st.restarts;
    p.B = B; p.H = H; p.Hkv = Hkv; p.S = S; p.causal = causal; p.lambda = lambda; p.mode = mode; p.c = c;
    p.b0_last = (b0_last && mode == BAPS_MODE_E2E_HIF8) ? 1 : 0;
    p.q_scale = q_scale; p.k_scale = k_scale;
    p.nq = S / 128; p.npairs = p.b0_last ? p.nq : (p.nq + 1) / 2;
    const long long nblocks = (long long)p.npairs * B * H;
    if (nblocks > 0x7fffffffLL) return BAPS_ERR_UNSUPPORTED;
    auto launch = [&](auto kernel, int sm) -> baps_status {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, sm) != cudaSuccess)
            return BAPS_ERR_CUDA;
        kernel<<<(unsigned)nblocks, kTcThreads, sm, stream>>>(mq, mk, mv, p);
        return launch_status();
    };
    constexpr int kE2E = BAPS_MODE_E2E_HIF8, kExact = BAPS_MODE_EXACT, kExp2m = BAPS_MODE_EXP2_HIF8;
    const bool b0l = p.b0_last != 0;
    if (qk8) {
        if (D != 128) return BAPS_ERR_UNSUPPORTED;
        if (mode == kExp2m) return launch(attention_tc_kernel<128, kExp2m, true, false>, TcLayout<128>::kDynBytes);
        if (mode == kExact) return launch(attention_tc_kernel<128, kExact, true, false>, TcLayout<128>::kDynBytes);
        return b0l ? launch(attention_tc_kernel<128, kE2E, true, true>, TcLayout<128>::kDynBytes)
                   : launch(attention_tc_kernel<128, kE2E, true, false>, TcLayout<128>::kDynBytes);
    }
    if (D == 128) {
        if (mode == kExp2m) return launch(attention_tc_kernel<128, kExp2m, false, false>, TcLayout<128>::kDynBytes);
        if (mode == kExact) return launch(attention_tc_kernel<128, kExact, false, false>, TcLayout<128>::kDynBytes);
        return b0l ? launch(attention_tc_kernel<128, kE2E, false, true>, TcLayout<128>::kDynBytes)
                   : launch(attention_tc_kernel<128, kE2E, false, false>, TcLayout<128>::kDynBytes);
    }
    if (mode == kExp2m) return launch(attention_tc_kernel<64, kExp2m, false, false>, TcLayout<64>::kDynBytes);
    if (mode == kExact) return launch(attention_tc_kernel<64, kExact, false, false>, TcLayout<64>::kDynBytes);
    return b0l ? launch(attention_tc_kernel<64, kE2E, false, true>, TcLayout<64>::kDynBytes)
               : launch(attention_tc_kernel<64, kE2E, false, false>, TcLayout<64>::kDynBytes);
}

} // namespace baps
