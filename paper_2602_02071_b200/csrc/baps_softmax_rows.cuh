// Row softmax by Algorithm 1 with one query row per "tile" and no value product (the
// non-fused path).  One CTA owns one row at a time:
//   pass 1  read the row from HBM, reduce the maximum of every block_k block into shared memory;
//   scan    one warp walks the blocks in order and applies the max bookkeeping of Algorithm 1
//           (block 0: m = ceil(max); later blocks: T = HiF8(max - m), restart if T > lambda,
//           else m += max(0, ceil(T))).  The state is one integer per row and only changes
//           at blocks whose maximum exceeds it, so the warp tests 32 blocks per ballot;
//   pass 2  re-read the row (it is still in L2), form the 8-bit weights, reduce d;
//   pass 3  re-read, form the weights again and write p = w * 2^(m_block - m_final) / d.
// HBM traffic is one read and one write of the row (8 bytes per element); the two re-reads are
// served by the 126 MB L2 because the rows in flight (one per CTA) are far smaller than it.
#pragma once
#include "baps_common.cuh"
#include "baps_hif8.cuh"

namespace baps {

constexpr int kSrThreads = 256;
constexpr int kSrMaxBlocks = 1024;     // 65536 / 64

// Max bookkeeping of Algorithm 1 for one block of a single row: given the running max m
// (integer valued, or -inf before block 0) and the block's largest logit xmax (base-2 score
// xmax * log2(e)), return the new max.  *restart is set when the restart branch was taken.
// T of the maximum is formed exactly as for every other element (one fused multiply-add).
__device__ __forceinline__ float row_block_update(float m, float xmax, bool first, int lambda,
                                                  bool *restart, float *delta)
{
    *restart = false; *delta = 0.f;
    if (first) return fmaxf(m, ceilf(xmax * kLog2e));
    const float t8 = hif8_round(fmaf(xmax, kLog2e, -m));
    if (t8 > (float)lambda) { *restart = true; return fmaxf(m, ceilf(xmax * kLog2e)); }
    const float d = fmaxf(0.f, ceilf(t8));
    *delta = d;
    return m + d;
}

template <int BK>
__global__ void __launch_bounds__(kSrThreads)
softmax_rows_kernel(const float *__restrict__ logits, float *__restrict__ probs, int64_t rows,
                    int cols, int lambda)
{
    __shared__ float s_bmax[kSrMaxBlocks];     // block maxima of the logits
    __shared__ float s_mbefore[kSrMaxBlocks];  // running max before each block (m~)
    __shared__ float s_lut[kLutN];
    __shared__ float s_red[kSrThreads / 32];
    __shared__ float s_mfinal, s_dinv;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int kWarps = kSrThreads / 32;
    constexpr int LPB = BK / 4;                // lanes per block (float4 per lane)
    constexpr int BPW = 32 / LPB;              // blocks per warp step (1 for 128, 2 for 64)
    const int nb = cols / BK;
    const int nchunks = cols / 128;            // a warp step covers 128 elements

    for (int i = tid; i < kLutN; i += kSrThreads) s_lut[i] = w0_table_entry(i);
    __syncthreads();

    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const float4 *x4 = reinterpret_cast<const float4 *>(logits + row * cols);
        float4 *p4 = reinterpret_cast<float4 *>(probs + row * cols);

        // ---- pass 1: block maxima -------------------------------------------------------
        for (int ch = warp; ch < nchunks; ch += kWarps) {
            const float4 v = __ldg(x4 + ch * 32 + lane);
            float mx = fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w));
#pragma unroll
            for (int o = LPB / 2; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            if ((lane % LPB) == 0) s_bmax[ch * BPW + lane / LPB] = mx;
        }
        __syncthreads();

        // ---- scan over blocks (warp 0) ---------------------------------------------------
        if (warp == 0) {
            bool rs; float dl;
            float m = row_block_update(-INFINITY, s_bmax[0], true, lambda, &rs, &dl);
            if (lane == 0) s_mbefore[0] = -INFINITY;
            for (int base = 1; base < nb; base += 32) {
                const int j = base + lane;
                const bool valid = j < nb;
                const float mj = valid ? s_bmax[j] : -INFINITY;
                bool pending = valid;
                while (true) {
                    const bool pred = pending && hif8_round(fmaf(mj, kLog2e, -m)) > 0.f;
                    const unsigned b = __ballot_sync(0xffffffffu, pred);
                    if (b == 0u) { if (pending) s_mbefore[j] = m; break; }
                    const int l = __ffs(b) - 1;
                    if (pending && lane <= l) { s_mbefore[j] = m; pending = false; }
                    const float ml = __shfl_sync(0xffffffffu, mj, l);
                    m = row_block_update(m, ml, false, lambda, &rs, &dl);
                }
            }
            if (lane == 0) s_mfinal = m;
        }
        __syncthreads();
        const float mfinal = s_mfinal;

        // ---- pass 2 / pass 3 ---------------------------------------------------------------
        float dsum = 0.f;
#pragma unroll 1
        for (int pass = 0; pass < 2; ++pass) {
            const float dinv = pass ? s_dinv : 0.f;
            for (int ch = warp; ch < nchunks; ch += kWarps) {
                const int j = ch * BPW + lane / LPB;
                const float4 v = __ldg(x4 + ch * 32 + lane);
                bool rs; float dl;
                const float mb = s_mbefore[j];
                const float ma = row_block_update(mb, s_bmax[j], j == 0, lambda, &rs, &dl);
                // weights of this block relative to ma, then moved to the final max
                const float shift = exp2f(ma - mfinal);      // exact power of two
                float w[4];
                const float xs[4] = {v.x, v.y, v.z, v.w};
                if (j == 0) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) w[e] = exp2f(fmaf(xs[e], kLog2e, -ma));
                } else {
                    const float mref = rs ? ma : mb;          // restart: T relative to the new max
                    const float post = rs ? 1.f : exp2f(-dl); // no restart: weights times 2^-delta
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        w[e] = s_lut[w0_index(fmaf(xs[e], kLog2e, -mref))] * post;
                }
                if (pass == 0) {
                    dsum += ((w[0] + w[1]) + (w[2] + w[3])) * shift;
                } else {
                    const float f = shift * dinv;
                    __stcs(p4 + ch * 32 + lane, make_float4(w[0] * f, w[1] * f, w[2] * f, w[3] * f));
                }
            }
            if (pass == 0) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, o);
                if (lane == 0) s_red[warp] = dsum;
                __syncthreads();
                if (tid == 0) {
                    float t = 0.f;
                    for (int i = 0; i < kWarps; ++i) t += s_red[i];
                    s_dinv = 1.f / t;
                }
                __syncthreads();
            }
        }
        __syncthreads();   // s_bmax / s_mbefore are reused by the next row
    }
}

} // namespace baps
