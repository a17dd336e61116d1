// Fused attention forward on the CUDA cores with float32 inputs: Algorithm 1 tile by tile, the
// scores accumulated in double precision.  This is the small-problem path (the single-head
// S = 128, D = 64 configuration) and the in-library cross-check of the tensor-core kernel; it
// makes no attempt at speed.  One CTA of 256 threads owns one query tile:
//   A  S = Q_i K_j^T * log2(e) * scale, masked entries -inf            (Algorithm 1, line S / T)
//   B  row maxima; tile-wide restart test on the 8-bit T               (restart condition)
//   C  max update, weights (fp32 2^x in the B0 tile, HiF8 table else)  (lines m, P)
//   D  d and O~ rescaled by exact powers of two and accumulated        (lines d, O~)
// and finally O = O~ / d.
#pragma once
#include "baps_common.cuh"
#include "baps_hif8.cuh"

namespace baps {

struct AttnF32Params {
    const float *q, *k, *v;
    float *out;                 // may be null
    float *row_m, *row_d, *out_f32;
    int32_t *restarts;
    int B, H, Hkv, S, D, causal, lambda, mode;
    int b0_last;                // B0 = {first, last visible key tile}: order 0, last, 1, ..., last - 1
    double c;                   // log2(e) * scale
};

constexpr int kAfThreads = 256;

template <int BQ, int BK>
__global__ void __launch_bounds__(kAfThreads)
attention_f32_kernel(const AttnF32Params p)
{
    extern __shared__ float smem[];
    float *s_S = smem;                         // [BQ][BK] scores, then weights
    float *s_m = s_S + BQ * BK;                // [BQ] running max
    float *s_d = s_m + BQ;                     // [BQ] denominator
    float *s_alpha = s_d + BQ;                 // [BQ] rescale of the previous state
    float *s_lut = s_alpha + BQ;               // [kLutN]
    __shared__ int s_flag;
    __shared__ int s_restarts;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int i0 = blockIdx.x * BQ, h = blockIdx.y, b = blockIdx.z;
    const int D = p.D, S = p.S;
    const int hk = h / (p.H / p.Hkv);
    const float *qh = p.q + ((size_t)b * p.H + h) * (size_t)S * D;
    const float *kh = p.k + ((size_t)b * p.Hkv + hk) * (size_t)S * D;
    const float *vh = p.v + ((size_t)b * p.Hkv + hk) * (size_t)S * D;

    for (int i = tid; i < kLutN; i += kAfThreads) s_lut[i] = w0_table_entry(i);
    for (int r = tid; r < BQ; r += kAfThreads) { s_m[r] = -INFINITY; s_d[r] = 0.f; }
    if (tid == 0) s_restarts = 0;

    // output accumulators: TPR threads per row, each owns columns t = sub + TPR * i
    constexpr int TPR = kAfThreads / BQ;
    constexpr int MAXC = 128 / TPR;
    const int orow = tid / TPR, osub = tid % TPR;
    float acc[MAXC];
#pragma unroll
    for (int i = 0; i < MAXC; ++i) acc[i] = 0.f;
    __syncthreads();

    const int jmax = p.causal ? (i0 + BQ - 1) / BK + 1 : S / BK;
    const bool order_last = p.b0_last && p.mode == BAPS_MODE_E2E_HIF8;
    const int nb0 = (order_last && jmax >= 2) ? 2 : 1;          // number of high-precision tiles
    for (int step = 0; step < jmax; ++step) {
        const int j = !order_last ? step : (step == 0 ? 0 : (step == 1 ? jmax - 1 : step - 1));
        const int c0 = j * BK;
        // ---- A: scores ---------------------------------------------------------------------
        for (int idx = tid; idx < BQ * BK; idx += kAfThreads) {
            const int r = idx / BK, cc = idx % BK;
            const float4 *qr = reinterpret_cast<const float4 *>(qh + (size_t)(i0 + r) * D);
            const float4 *kc = reinterpret_cast<const float4 *>(kh + (size_t)(c0 + cc) * D);
            double a = 0.0;
            for (int t = 0; t < D / 4; ++t) {
                const float4 x = __ldg(qr + t), y = __ldg(kc + t);
                a += (double)x.x * y.x; a += (double)x.y * y.y;
                a += (double)x.z * y.z; a += (double)x.w * y.w;
            }
            float s = (float)(a * p.c);
            if (p.causal && c0 + cc > i0 + r) s = -INFINITY;
            s_S[idx] = s;
        }
        if (tid == 0) s_flag = 0;
        __syncthreads();
        const bool hp = (step < nb0 && p.mode != BAPS_MODE_EXP2_HIF8) || (p.mode == BAPS_MODE_EXACT);   // high-precision tile
        // ---- B: restart test (one decision per tile) ----------------------------------------
        if (!hp && p.mode != BAPS_MODE_EXP2_HIF8) {
            for (int r = warp; r < BQ; r += kAfThreads / 32) {
                float mx = -INFINITY;
                for (int cc = lane; cc < BK; cc += 32) mx = fmaxf(mx, s_S[r * BK + cc]);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                if (lane == 0 && hif8_round(mx - s_m[r]) > (float)p.lambda) s_flag = 1;
            }
            __syncthreads();
        }
        const bool restart = !hp && p.mode != BAPS_MODE_EXP2_HIF8 && s_flag != 0;
        if (tid == 0 && restart) ++s_restarts;
        // ---- C: max update and weights -------------------------------------------------------
        for (int r = warp; r < BQ; r += kAfThreads / 32) {
            float mx = -INFINITY;
            for (int cc = lane; cc < BK; cc += 32) mx = fmaxf(mx, s_S[r * BK + cc]);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            const float mold = s_m[r];
            float mnew, alpha, sum = 0.f;
            if (p.mode == BAPS_MODE_EXACT) {
                mnew = fmaxf(mold, mx);                              // Eq. (2): real-valued max
                alpha = (mold == -INFINITY) ? 0.f : exp2f(mold - mnew);
                for (int cc = lane; cc < BK; cc += 32) {
                    const float w = (mnew == -INFINITY) ? 0.f : exp2f(s_S[r * BK + cc] - mnew);
                    s_S[r * BK + cc] = w; sum += w;
                }
            } else if (p.mode == BAPS_MODE_EXP2_HIF8) {
                // "Exp2 HiF8" setup (Section 4.1): Eq. (2) with every 2^x through Algorithm 2
                mnew = fmaxf(mold, mx);
                alpha = (mold == -INFINITY) ? 0.f : s_lut[w0_index(mold - mnew)];
                for (int cc = lane; cc < BK; cc += 32) {
                    const float w = (mnew == -INFINITY) ? 0.f : s_lut[w0_index(s_S[r * BK + cc] - mnew)];
                    s_S[r * BK + cc] = w; sum += w;
                }
            } else if (hp || restart) {
                mnew = fmaxf(mold, ceilf(mx));
                alpha = (mold == -INFINITY) ? 0.f : exp2f(mold - mnew);
                for (int cc = lane; cc < BK; cc += 32) {
                    const float u = s_S[r * BK + cc] - mnew;
                    const float w = hp ? ((mnew == -INFINITY) ? 0.f : exp2f(u)) : s_lut[w0_index(u)];
                    s_S[r * BK + cc] = w; sum += w;
                }
            } else {
                const float t8 = hif8_round(mx - mold);
                const float delta = fmaxf(0.f, ceilf(t8));           // 0 for an all-masked row
                mnew = mold + delta;
                alpha = exp2f(-delta);
                for (int cc = lane; cc < BK; cc += 32) {
                    const float w = s_lut[w0_index(s_S[r * BK + cc] - mold)] * alpha;
                    s_S[r * BK + cc] = w; sum += w;
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (lane == 0) { s_m[r] = mnew; s_alpha[r] = alpha; s_d[r] = alpha * s_d[r] + sum; }
        }
        __syncthreads();
        // ---- D: O~ = alpha O~ + W V_j ---------------------------------------------------------
        {
            const float al = s_alpha[orow];
#pragma unroll
            for (int i = 0; i < MAXC; ++i) acc[i] *= al;
            for (int cc = 0; cc < BK; ++cc) {
                const float w = s_S[orow * BK + cc];
                if (w == 0.f) continue;
                const float *vr = vh + (size_t)(c0 + cc) * D;
#pragma unroll
                for (int i = 0; i < MAXC; ++i) {
                    const int t = osub + TPR * i;
                    if (t < D) acc[i] = fmaf(w, __ldg(vr + t), acc[i]);
                }
            }
        }
        __syncthreads();
    }
    // ---- normalisation and statistics ------------------------------------------------------------
    {
        const float dinv = 1.f / s_d[orow];
        const size_t rowoff = (((size_t)b * p.H + h) * S + (i0 + orow)) * (size_t)D;
#pragma unroll
        for (int i = 0; i < MAXC; ++i) {
            const int t = osub + TPR * i;
            if (t < D) {
                const float o = acc[i] * dinv;
                if (p.out) p.out[rowoff + t] = o;
                if (p.out_f32) p.out_f32[rowoff + t] = o;
            }
        }
    }
    const size_t srow = ((size_t)b * p.H + h) * S + i0;
    for (int r = tid; r < BQ; r += kAfThreads) {
        if (p.row_m) p.row_m[srow + r] = s_m[r];
        if (p.row_d) p.row_d[srow + r] = s_d[r];
    }
    if (tid == 0 && p.restarts)
        p.restarts[((size_t)b * p.H + h) * (S / BQ) + blockIdx.x] = s_restarts;
}

template <int BQ, int BK>
constexpr size_t attention_f32_smem() { return sizeof(float) * (BQ * BK + 3 * BQ + kLutN); }

} // namespace baps
