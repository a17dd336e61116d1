// Row softmax by Algorithm 1 with one query row per "tile" and no value product (the
// non-fused path).  One CTA owns one row at a time:
//   pass 1  read the row from HBM, reduce the maximum of every block_k block into shared memory;
//   scan    one warp walks the blocks in order and applies the max bookkeeping of Algorithm 1
//           (block 0: m = ceil(max); later blocks: T = HiF8(max - m), restart if T > lambda,
//           else m += max(0, ceil(T))).  The state is one integer per row and only changes
//           at blocks whose maximum exceeds it, so the warp tests 32 blocks per ballot;
//   pass 2  form the 8-bit weights, reduce d;
//   pass 3  write p = w * 2^(m_block - m_final) / d.
// Rows of 1K columns are handled by one warp each (softmax_rows_warp_kernel), rows of 2K, 4K and 8K
// columns by groups of threads that share a CTA and its tables (softmax_rows_group_kernel), rows of 16K
// and 32K by one CTA each, fed through a shared-memory ring by bulk asynchronous copies so that the read
// of the next row overlaps the passes over the current one, rows of 64K by one CTA that keeps half the row
// in registers and half in the shared-memory pieces it arrived in.  In all of these the row stays on chip
// between the passes, so HBM traffic is exactly one read and one write of the row (8 bytes per element).  Other lengths use the generic variant, which re-reads
// the row from L2 in passes 2 and 3.
// Blocks whose T are all <= 0 (nearly all of them) take the weights from a bank-replicated table keyed
// by the top bits of -T * 2^-120, as the fused attention kernel does.  What a block's weights need --
// the max its T are taken against, the power of two that moves them to the final max, which table --
// is worked out once per block by one lane and handed round by shuffles.
#pragma once
#include "baps_common.cuh"
#include "baps_hif8.cuh"
#include "baps_tables.cuh"
#include "baps_sm100.cuh"

namespace baps {

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
    const float u = fmaf(xmax, kLog2e, -m);
    if (u <= 0.f) return m;                     // T8 <= 0: no restart, delta = 0 (the common case)
    const float t8 = hif8_round(u);
    if (t8 > (float)lambda) { *restart = true; return fmaxf(m, ceilf(xmax * kLog2e)); }
    const float d = fmaxf(0.f, ceilf(t8));
    *delta = d;
    return m + d;
}

// Maximum over the LPB lanes that hold one block.  LPB = 32 (the whole warp): one reduction instruction
// (REDUX) or five shuffles -- which of the two is faster depends on the kernel around it (measured: the
// instruction wins by 5 to 10 % in most variants and loses as much in the 4K-column group variant and the
// 16K-column ring variant), so the callers choose.  LPB = 16: the two halves of the warp, by shuffles.
template <int LPB, bool REDUX = true>
__device__ __forceinline__ float lanes_max(float mx)
{
    if constexpr (LPB == 32 && REDUX) {
        float r;
        asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(mx));
        return r;
    } else {
#pragma unroll
        for (int o = LPB / 2; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        return mx;
    }
}

// What the weights pass needs to know about one block, worked out once per block (by one lane) and
// handed to the lanes that hold the block's elements by a shuffle: the max its T are taken against,
// the exact power of two that moves its weights to the row's final max (2^-delta included), and how
// the weights are formed: 0 = block 0 (high precision), 1 = every T <= 0 (bank-replicated table keyed
// by the top bits), 2 = the block holds a positive T (full table).
struct BlockParams { float mref, scale; int kind; };

__device__ __forceinline__ BlockParams block_params(float mb, float bm, bool first, int lambda, float mfinal)
{
    bool rs; float dl;
    const float ma = row_block_update(mb, bm, first, lambda, &rs, &dl);
    BlockParams p;
    p.mref = (first || rs) ? ma : mb;          // restart / block 0: the new max; otherwise the old one,
    p.scale = exp2f(p.mref - mfinal);          // and then 2^-delta 2^(m_after - m_final) = 2^(m_before - m_final)
    p.kind = first ? 0 : (fmaf(bm, kLog2e, -p.mref) > 0.f ? 2 : 1);
    return p;
}

// Weights of one 16-byte vector of a block, already moved to the final max.  any_pos: some block of
// this warp-wide vector holds a positive T (warp-uniform for BK = 128), in which case the whole vector
// takes the full table.
template <bool FAST>
__device__ __forceinline__ float4 block_weights(const float4 &x, float mref, float scale, int kind, bool any_pos,
                                                const float *s_rep, const float *s_lut, int lane)
{
    float4 w;
    if (kind == 0) {
        w.x = exp2f(fmaf(x.x, kLog2e, -mref)); w.y = exp2f(fmaf(x.y, kLog2e, -mref));
        w.z = exp2f(fmaf(x.z, kLog2e, -mref)); w.w = exp2f(fmaf(x.w, kLog2e, -mref));
    } else if (FAST && !any_pos) {
        // x = -T * 2^-120 by one fused multiply-add with flush-to-zero (|T| < 2^-6 becomes +0, weight
        // 1), the top bits of x select the entry (everything from |T| >= 32 on is the entry 0)
        const float cn = -kLog2e * 7.52316384526264e-37f, mn = mref * 7.52316384526264e-37f;   // 2^-120
        auto fast = [&](float xv) {
            float t;
            asm("fma.rn.ftz.f32 %0, %1, %2, %3;" : "=f"(t) : "f"(xv), "f"(cn), "f"(mn));
            return s_rep[min(__float_as_uint(t) >> 19, 192u) * 32u + lane];
        };
        w.x = fast(x.x); w.y = fast(x.y); w.z = fast(x.z); w.w = fast(x.w);
    } else {
        w.x = s_lut[w0_index(fmaf(x.x, kLog2e, -mref))]; w.y = s_lut[w0_index(fmaf(x.y, kLog2e, -mref))];
        w.z = s_lut[w0_index(fmaf(x.z, kLog2e, -mref))]; w.w = s_lut[w0_index(fmaf(x.w, kLog2e, -mref))];
    }
    return make_float4(w.x * scale, w.y * scale, w.z * scale, w.w * scale);
}

// The parameters of the NV * BPW blocks a warp holds, one block per lane (lane = BPW * k + q for block
// q of the warp's k-th vector); packed kind: bits 0-1 the block's kind, bit 2 "some block of the same
// vector holds a positive T".
template <int BPW>
__device__ __forceinline__ int pack_kind(int kind)
{
    int slow = kind == 2;
    if (BPW == 2) slow |= __shfl_xor_sync(0xffffffffu, kind, 1) == 2;
    return kind | (slow << 2);
}

// The scan of Algorithm 1's max bookkeeping over the NB block maxima of one row, by one warp: writes the
// running max before every block and the final max.  The state is one integer per row and only changes at
// blocks whose maximum exceeds it, so the warp tests 32 blocks per ballot.  (The loop over the groups of
// 32 blocks is kept rolled: unrolled, with the inner loop and the update inlined four or more times, the
// same kernel ran 20 % slower.)
template <int NB>
__device__ __forceinline__ void scan_blocks(const float *s_bmax, float *s_mbefore, float *s_mfinal, int lambda, int lane)
{
    bool rs; float dl;
    float m = row_block_update(-INFINITY, s_bmax[0], true, lambda, &rs, &dl);
    if (lane == 0) s_mbefore[0] = -INFINITY;
#pragma unroll 1
    for (int base = 1; base < NB; base += 32) {
        const int j = base + lane;
        const bool valid = j < NB;
        const float mj = valid ? s_bmax[j] : -INFINITY;
        bool pending = valid;
        while (true) {
            // HiF8(T) > 0  <=>  T >= 2^-23 (smaller magnitudes round to zero)
            const bool pred = pending && fmaf(mj, kLog2e, -m) >= 1.1920928955078125e-07f;
            const unsigned b = __ballot_sync(0xffffffffu, pred);
            if (b == 0u) { if (pending) s_mbefore[j] = m; break; }
            const int l = __ffs(b) - 1;
            if (pending && lane <= l) { s_mbefore[j] = m; pending = false; }
            const float ml = __shfl_sync(0xffffffffu, mj, l);
            m = row_block_update(m, ml, false, lambda, &rs, &dl);
        }
    }
    if (lane == 0) *s_mfinal = m;
}

// Bulk asynchronous copy of one row (or part of one) into shared memory, completion counted on an
// mbarrier: in pieces of at most 32 KB, all on the same barrier.
__device__ __forceinline__ void bulk_load_row(uint32_t dst, const float *src, uint32_t bytes, uint32_t bar)
{
    for (uint32_t off = 0; off < bytes; off += 32768u) {
        const uint32_t n = bytes - off < 32768u ? bytes - off : 32768u;
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(dst + off), "l"(reinterpret_cast<const float *>(src) + off / 4), "r"(n), "r"(bar)
                     : "memory");
    }
}

// Any row length that is a multiple of 128 (the lengths without a kernel of their own): one CTA per row
// at a time, the row is read three times -- from HBM for the block maxima, then again (from L2) for the
// sum of the weights and for the output.  BK: block size of Algorithm 1 along the row (64 or 128).
// FAST: blocks without a positive T use the bank-replicated table (25 KB of shared memory).
template <int BK, int THREADS, bool FAST>
__global__ void __launch_bounds__(THREADS)
softmax_rows_generic_kernel(const float *__restrict__ logits, float *__restrict__ probs, int64_t rows,
                            int cols, int lambda)
{
    __shared__ float s_bmax[kSrMaxBlocks];     // block maxima of the logits
    __shared__ float s_mbefore[kSrMaxBlocks];  // running max before each block (m~)
    __shared__ float s_lut[kLutN];
    __shared__ __align__(16) float s_rep[FAST ? (16 + kLutNegN) * 32 : 32];
    __shared__ float s_red[THREADS / 32];
    __shared__ float s_mfinal;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int kWarps = THREADS / 32;
    constexpr int LPB = BK / 4;                // lanes per block (float4 per lane)
    constexpr int BPW = 32 / LPB;              // blocks per warp step (1 for 128, 2 for 64)
    const int nb = cols / BK;
    const int nchunks = cols / 128;            // a warp step covers 128 elements

    for (int i = tid; i < kLutN; i += THREADS) s_lut[i] = g_w0_table[i];
    for (int e = tid; FAST && e < 16 + kLutNegN; e += THREADS) {
        const float w = (e < 16) ? 1.f : g_w0_table[e - 16];
        const float4 w4 = make_float4(w, w, w, w);
#pragma unroll
        for (int i = 0; i < 8; ++i) reinterpret_cast<float4 *>(s_rep)[e * 8 + i] = w4;
    }
    __syncthreads();

    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const float4 *x4 = reinterpret_cast<const float4 *>(logits + row * cols);
        float4 *p4 = reinterpret_cast<float4 *>(probs + row * cols);
        // ---- pass 1: block maxima (the only HBM read of the row) ----------------------------------------
        for (int ch = warp; ch < nchunks; ch += kWarps) {
            const float4 x = __ldg(x4 + ch * 32 + lane);
            float mx = fmaxf(fmaxf(x.x, x.y), fmaxf(x.z, x.w));
            mx = lanes_max<LPB>(mx);
            if ((lane % LPB) == 0) s_bmax[ch * BPW + lane / LPB] = mx;
        }
        __syncthreads();
        // ---- scan over the blocks (warp 0) ---------------------------------------------------------------
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
                    // HiF8(T) > 0  <=>  T >= 2^-23 (smaller magnitudes round to zero)
                    const bool pred = pending && fmaf(mj, kLog2e, -m) >= 1.1920928955078125e-07f;
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
        // weights of one 16-byte vector, already moved to the final max
        auto weights = [&](const float4 &x, int ch) {
            const int j = ch * BPW + lane / LPB;
            const BlockParams bp = block_params(s_mbefore[j], s_bmax[j], j == 0, lambda, mfinal);
            // some lane of the warp holds a block with a positive T: voted by the whole warp
            const bool any_pos = __any_sync(0xffffffffu, bp.kind == 2);
            return block_weights<FAST>(x, bp.mref, bp.scale, bp.kind, any_pos, s_rep, s_lut, lane);
        };
        // ---- pass 2: the sum of the weights ----------------------------------------------------------------
        float dsum = 0.f;
        for (int ch = warp; ch < nchunks; ch += kWarps) {
            const float4 w = weights(__ldg(x4 + ch * 32 + lane), ch);
            dsum += (w.x + w.y) + (w.z + w.w);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, o);
        if (lane == 0) s_red[warp] = dsum;
        __syncthreads();
        float t = 0.f;                          // every thread adds the partial sums itself, in the same order
#pragma unroll
        for (int i = 0; i < kWarps; ++i) t += s_red[i];
        const float dinv = 1.f / t;
        // ---- pass 3: p = w * 2^(m_block - m_final) / d -----------------------------------------------------
        for (int ch = warp; ch < nchunks; ch += kWarps) {
            const float4 w = weights(__ldg(x4 + ch * 32 + lane), ch);
            __stcs(p4 + ch * 32 + lane, make_float4(w.x * dinv, w.y * dinv, w.z * dinv, w.w * dinv));
        }
        __syncthreads();   // s_bmax / s_mbefore / s_red are reused by the next row
    }
}

// Table words of the 8-bit-output kernels: the fp32 pattern of w0(T) with its HiF8 code in the low byte.
__device__ __forceinline__ uint32_t w0_word(float w) { return __float_as_uint(w) | (uint32_t)hif8_pack(w); }

// Parameters of one block for the 8-bit output: the max its T are taken against (block 0 is no exception
// here), the integer exponent of the block, and whether the block holds a positive T (kind 2) or not (1).
struct CodesBlockParams { float mref; int bexp; int kind; float scale; };   // scale = 2^bexp
__device__ __forceinline__ CodesBlockParams codes_block_params(float mb, float bm, bool first, int lambda, float mfinal)
{
    bool rs; float dl;
    const float ma = row_block_update(mb, bm, first, lambda, &rs, &dl);
    CodesBlockParams p;
    p.mref = (first || rs) ? ma : mb;
    p.bexp = (int)(p.mref - mfinal);
    p.scale = exp2f(p.mref - mfinal);
    p.kind = fmaf(bm, kLog2e, -p.mref) > 0.f ? 2 : 1;
    return p;
}

// Table words of one 16-byte vector.
template <bool FAST>
__device__ __forceinline__ uint4 block_words(const float4 &x, float mref, bool any_pos, const uint32_t *s_rep,
                                             const uint32_t *s_lut, int lane)
{
    uint4 e;
    if (FAST && !any_pos) {
        const float cn = -kLog2e * 7.52316384526264e-37f, mn = mref * 7.52316384526264e-37f;   // 2^-120
        auto fast = [&](float xv) {
            float t;
            asm("fma.rn.ftz.f32 %0, %1, %2, %3;" : "=f"(t) : "f"(xv), "f"(cn), "f"(mn));
            return s_rep[min(__float_as_uint(t) >> 19, 192u) * 32u + lane];
        };
        e.x = fast(x.x); e.y = fast(x.y); e.z = fast(x.z); e.w = fast(x.w);
    } else {
        e.x = s_lut[w0_index(fmaf(x.x, kLog2e, -mref))]; e.y = s_lut[w0_index(fmaf(x.y, kLog2e, -mref))];
        e.z = s_lut[w0_index(fmaf(x.z, kLog2e, -mref))]; e.w = s_lut[w0_index(fmaf(x.w, kLog2e, -mref))];
    }
    return e;
}

// Where a row kernel writes: probabilities (float output), or codes, block exponents and denominators
// (8-bit output; see the description further down).
struct RowsOut {
    float *probs;
    uint8_t *codes;
    int32_t *block_exp;
    float *row_d;
};

// Tables of a CTA in shared memory, as words: float output keeps the fp32 pattern of w0, 8-bit output the
// pattern with the HiF8 code in its low byte.
template <bool CODES, int NTHREADS>
__device__ __forceinline__ void fill_tables(uint32_t *s_lut, uint32_t *s_rep, int t)
{
    for (int i = t; i < kLutN; i += NTHREADS) s_lut[i] = CODES ? w0_word(g_w0_table[i]) : __float_as_uint(g_w0_table[i]);
    for (int e = t; e < 16 + kLutNegN; e += NTHREADS) {
        const float w = (e < 16) ? 1.f : g_w0_table[e - 16];
        const uint32_t u = CODES ? w0_word(w) : __float_as_uint(w);
        const uint4 u4 = make_uint4(u, u, u, u);
#pragma unroll
        for (int i = 0; i < 8; ++i) reinterpret_cast<uint4 *>(s_rep)[e * 8 + i] = u4;
    }
}

// 8-bit output of one vector: its table words -> four codes (stored), returns the sum of the decoded weights
// times the block's scale 2^bexp.
__device__ __forceinline__ float emit_codes(uint32_t *dst, const uint4 &e, float scale)
{
    __stcs(dst, (e.x & 0xFFu) | ((e.y & 0xFFu) << 8) | ((e.z & 0xFFu) << 16) | (e.w << 24));
    return ((__uint_as_float(e.x & 0xFFFFFF00u) + __uint_as_float(e.y & 0xFFFFFF00u)) +
            (__uint_as_float(e.z & 0xFFFFFF00u) + __uint_as_float(e.w & 0xFFFFFF00u))) * scale;
}

// Long rows (16K, 32K columns): one CTA per row at a time with the row in registers (32 floats per
// thread: 512 threads for 16K, two CTAs per SM; 1024 threads for 32K), fed through a one-row
// shared-memory ring by bulk asynchronous copies (cp.async.bulk, completion on an mbarrier) that one
// thread issues as soon as the current row sits in registers, i.e. after the first barrier of the row:
// the HBM read of the next row overlaps the scan, the weights and the write of the current one.
// Three barriers per row.  CODES: 8-bit output.
template <int BK, int THREADS, bool CODES, bool REDUX = true>
__global__ void __launch_bounds__(THREADS, 2048 / THREADS / 2)
softmax_rows_ring_kernel(const float *__restrict__ logits, RowsOut out, int64_t rows, int lambda)
{
    constexpr int NV = 8, kWarps = THREADS / 32, cols = NV * THREADS * 4;
    constexpr int LPB = BK / 4, BPW = 32 / LPB, nb = cols / BK;
    constexpr uint32_t row_bytes = (uint32_t)cols * 4u;
    static_assert(NV * BPW <= 32, "one block per lane");
    extern __shared__ __align__(128) uint8_t sr_ring[];          // one row
    __shared__ __align__(8) uint64_t s_full;
    __shared__ int s_abort;
    __shared__ float s_bmax[nb];
    __shared__ float s_mbefore[nb];
    __shared__ uint32_t s_lut[kLutN];
    __shared__ __align__(16) uint32_t s_rep[(16 + kLutNegN) * 32];
    __shared__ float s_red[kWarps];
    __shared__ float s_mfinal;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    fill_tables<CODES, THREADS>(s_lut, s_rep, tid);
    if (tid == 0) {
        sm100::mbar_init(sm100::smem_u32(&s_full), 1);
        sm100::mbar_fence_init();
        s_abort = 0;
    }
    __syncthreads();
    if (tid == 0 && (int64_t)blockIdx.x < rows) {
        sm100::mbar_arrive_expect_tx(sm100::smem_u32(&s_full), row_bytes);
        bulk_load_row(sm100::smem_u32(sr_ring), logits + (int64_t)blockIdx.x * cols, row_bytes, sm100::smem_u32(&s_full));
    }

    int it = 0;
    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x, ++it) {
        float4 v[NV];
        // ---- pass 1: the row into registers, block maxima ----------------------------------------------
        // bounded wait; after a time-out the kernel runs on (on stale data) so that every thread keeps
        // meeting the same barriers, and the status word reports the failure
        sm100::mbar_wait(sm100::smem_u32(&s_full), (uint32_t)(it & 1), &s_abort, &g_async_status, 0x400);
        {
            const float4 *ring4 = reinterpret_cast<const float4 *>(sr_ring);
#pragma unroll
            for (int k = 0; k < NV; ++k) v[k] = ring4[(warp + k * kWarps) * 32 + lane];
        }
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            float mx = fmaxf(fmaxf(v[k].x, v[k].y), fmaxf(v[k].z, v[k].w));
            mx = lanes_max<LPB, REDUX>(mx);
            if ((lane % LPB) == 0) s_bmax[(warp + k * kWarps) * BPW + lane / LPB] = mx;
        }
        __syncthreads();
        if (tid == 0) {
            const int64_t rn = row + gridDim.x;             // the ring takes the next row
            if (rn < rows) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                sm100::mbar_arrive_expect_tx(sm100::smem_u32(&s_full), row_bytes);
                bulk_load_row(sm100::smem_u32(sr_ring), logits + rn * cols, row_bytes, sm100::smem_u32(&s_full));
            }
        }
        // ---- scan over the blocks (warp 0) ---------------------------------------------------------------
        if (warp == 0) scan_blocks<nb>(s_bmax, s_mbefore, &s_mfinal, lambda, lane);
        __syncthreads();
        const float mfinal = s_mfinal;
        const int jmine = (warp + (lane / BPW) * kWarps) * BPW + lane % BPW;      // the block whose parameters I work out
        float dsum = 0.f;
        if constexpr (CODES) {
            // ---- pass 2: codes, block exponents, the sum of the decoded weights ---------------------------
            uint32_t *c4 = reinterpret_cast<uint32_t *>(out.codes + row * cols);
            CodesBlockParams bp = {0.f, 0, 1, 0.f};
            if (lane < NV * BPW) {
                bp = codes_block_params(s_mbefore[jmine], s_bmax[jmine], jmine == 0, lambda, mfinal);
                out.block_exp[row * nb + jmine] = bp.bexp;
            }
            const int kindp = pack_kind<BPW>(bp.kind);
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int src = k * BPW + lane / LPB;
                const float mref = __shfl_sync(0xffffffffu, bp.mref, src);
                const float be = __shfl_sync(0xffffffffu, bp.scale, src);
                const int kp = __shfl_sync(0xffffffffu, kindp, src);
                dsum += emit_codes(c4 + (warp + k * kWarps) * 32 + lane,
                                   block_words<true>(v[k], mref, (kp & 4) != 0, s_rep, s_lut, lane), be);
            }
        } else {
            // ---- pass 2: weights (already moved to the final max) and their sum ---------------------------
            BlockParams bp = {0.f, 0.f, 1};
            if (lane < NV * BPW) bp = block_params(s_mbefore[jmine], s_bmax[jmine], jmine == 0, lambda, mfinal);
            const int kindp = pack_kind<BPW>(bp.kind);
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int src = k * BPW + lane / LPB;
                const float mref = __shfl_sync(0xffffffffu, bp.mref, src), scale = __shfl_sync(0xffffffffu, bp.scale, src);
                const int kp = __shfl_sync(0xffffffffu, kindp, src);
                v[k] = block_weights<true>(v[k], mref, scale, kp & 3, (kp & 4) != 0, reinterpret_cast<const float *>(s_rep),
                                           reinterpret_cast<const float *>(s_lut), lane);
                dsum += (v[k].x + v[k].y) + (v[k].z + v[k].w);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, o);
        if (lane == 0) s_red[warp] = dsum;
        __syncthreads();
        if constexpr (CODES) {
            if (tid == 0) {
                float t = 0.f;
#pragma unroll
                for (int i = 0; i < kWarps; ++i) t += s_red[i];
                out.row_d[row] = t;
            }
        } else {
            // every thread adds the warps' partial sums itself, in the same order
            float t = 0.f;
#pragma unroll
            for (int i = 0; i < kWarps; ++i) t += s_red[i];
            const float dinv = 1.f / t;
            // ---- pass 3 ---------------------------------------------------------------------------------
            float4 *p4 = reinterpret_cast<float4 *>(out.probs + row * cols);
#pragma unroll
            for (int k = 0; k < NV; ++k)
                __stcs(p4 + (warp + k * kWarps) * 32 + lane,
                       make_float4(v[k].x * dinv, v[k].y * dinv, v[k].z * dinv, v[k].w * dinv));
        }
        // (no barrier here: what the next row writes first, s_bmax, was last read before the third barrier
        // above; s_mbefore, s_mfinal and s_red are written behind the next row's first and second barrier,
        // which every thread -- the one adding up s_red included -- joins only when it is done with this row)
    }
}

// Rows of 64K columns: one CTA of 1024 threads holds the whole row on chip, half in registers and half in
// shared memory (128 KB each -- neither alone could hold it), so HBM traffic stays one read and one write of
// the row and no barrier crosses SMs.  The row travels in four quarters of 16K columns (64 KB) through three
// shared-memory pieces.  Quarters 0 and 1 pass through the transit piece into registers (16 floats per thread
// each); quarters 2 and 3 stay in their pieces until the row is done with them (for the float output their
// weights are formed twice, for the sum and again for the output, rather than written back).  Every piece is
// requested again as soon as it is free: the transit piece takes quarter 1 once quarter 0 sits in registers and the
// next row's quarter 0 once quarter 1 does; the piece of quarter 2 takes the next row's quarter 2 when the
// output pass is through with it, likewise quarter 3 -- so of the next row only quarter 1 is waited for in
// the open.  Seven barriers per row.
template <int BK, bool CODES>
__global__ void __launch_bounds__(1024, 1)
softmax_rows_quarters_kernel(const float *__restrict__ logits, RowsOut out, int64_t rows, int lambda)
{
    constexpr int THREADS = 1024, NQ = 4, kWarps = THREADS / 32, kQuarter = NQ * THREADS * 4, cols = 4 * kQuarter;
    constexpr int LPB = BK / 4, BPW = 32 / LPB, nbq = kQuarter / BK, nb = 4 * nbq;
    constexpr uint32_t q_bytes = (uint32_t)kQuarter * 4u;
    static_assert(NQ * BPW <= 32, "one block per lane and quarter");
    extern __shared__ __align__(128) uint8_t sr_ring[];          // three pieces of one quarter row each
    __shared__ __align__(8) uint64_t s_full[3];
    __shared__ int s_abort;
    __shared__ float s_bmax[nb];
    __shared__ float s_mbefore[nb];
    __shared__ uint32_t s_lut[kLutN];
    __shared__ __align__(16) uint32_t s_rep[(16 + kLutNegN) * 32];
    __shared__ float s_red[kWarps];
    __shared__ float s_mfinal;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    fill_tables<CODES, THREADS>(s_lut, s_rep, tid);
    if (tid == 0) {
        for (int i = 0; i < 3; ++i) sm100::mbar_init(sm100::smem_u32(&s_full[i]), 1);
        sm100::mbar_fence_init();
        s_abort = 0;
    }
    __syncthreads();
    // one thread: piece `pc` takes quarter `q` of row `r`
    auto request = [&](int pc, int64_t r, int q) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        sm100::mbar_arrive_expect_tx(sm100::smem_u32(&s_full[pc]), q_bytes);
        bulk_load_row(sm100::smem_u32(sr_ring) + (uint32_t)pc * q_bytes, logits + r * cols + (int64_t)q * kQuarter, q_bytes,
                      sm100::smem_u32(&s_full[pc]));
    };
    if (tid == 0 && (int64_t)blockIdx.x < rows) {
        request(0, blockIdx.x, 0);
        request(1, blockIdx.x, 2);
        request(2, blockIdx.x, 3);
    }
    const float4 *piece[3] = {reinterpret_cast<const float4 *>(sr_ring), reinterpret_cast<const float4 *>(sr_ring + q_bytes),
                              reinterpret_cast<const float4 *>(sr_ring + 2 * q_bytes)};
    const float *f_rep = reinterpret_cast<const float *>(s_rep), *f_lut = reinterpret_cast<const float *>(s_lut);
    uint32_t ph0 = 0, ph1 = 0, ph2 = 0;         // phase parities of the three pieces (the same in every thread)
    // bounded waits; after a time-out the kernel runs on (on stale data) so that every thread keeps meeting
    // the same barriers, and the status word reports the failure
    auto wait_piece = [&](int pc, uint32_t &ph, int code) {
        sm100::mbar_wait(sm100::smem_u32(&s_full[pc]), ph & 1u, &s_abort, &g_async_status, code);
        ph ^= 1u;
    };
    auto block_max = [&](const float4 &x, int j0) {
        float mx = fmaxf(fmaxf(x.x, x.y), fmaxf(x.z, x.w));
        mx = lanes_max<LPB>(mx);
        if ((lane % LPB) == 0) s_bmax[j0 + lane / LPB] = mx;
    };
    const int vi0 = warp * 32 + lane;           // my vector k of a quarter is number vi0 + k * THREADS of it

    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const bool more = row + gridDim.x < rows;
        float4 v[2 * NQ];                       // quarters 0 and 1
        // ---- quarters 0 and 1: through the transit piece into registers, block maxima -----------------------
        wait_piece(0, ph0, 0x420);
#pragma unroll
        for (int k = 0; k < NQ; ++k) v[k] = piece[0][vi0 + k * THREADS];
        __syncthreads();
        if (tid == 0) request(0, row, 1);
#pragma unroll
        for (int k = 0; k < NQ; ++k) block_max(v[k], (warp + k * kWarps) * BPW);
        wait_piece(0, ph0, 0x421);
#pragma unroll
        for (int k = 0; k < NQ; ++k) v[NQ + k] = piece[0][vi0 + k * THREADS];
        __syncthreads();
        if (tid == 0 && more) request(0, row + gridDim.x, 0);
#pragma unroll
        for (int k = 0; k < NQ; ++k) block_max(v[NQ + k], nbq + (warp + k * kWarps) * BPW);
        // ---- quarters 2 and 3: stay in their pieces; block maxima -------------------------------------------
        wait_piece(1, ph1, 0x422);
#pragma unroll
        for (int k = 0; k < NQ; ++k) block_max(piece[1][vi0 + k * THREADS], 2 * nbq + (warp + k * kWarps) * BPW);
        wait_piece(2, ph2, 0x423);
#pragma unroll
        for (int k = 0; k < NQ; ++k) block_max(piece[2][vi0 + k * THREADS], 3 * nbq + (warp + k * kWarps) * BPW);
        __syncthreads();
        if (warp == 0) scan_blocks<nb>(s_bmax, s_mbefore, &s_mfinal, lambda, lane);
        __syncthreads();
        const float mfinal = s_mfinal;
        // the block of quarter qq whose parameters my lane works out (lane < NQ * BPW)
        const int jl = (warp + (lane / BPW) * kWarps) * BPW + lane % BPW;
        float dsum = 0.f;
        if constexpr (CODES) {
            uint32_t *c4 = reinterpret_cast<uint32_t *>(out.codes + row * cols);
#pragma unroll
            for (int qq = 0; qq < 4; ++qq) {
                CodesBlockParams bp = {0.f, 0, 1, 0.f};
                if (lane < NQ * BPW) {
                    const int j = qq * nbq + jl;
                    bp = codes_block_params(s_mbefore[j], s_bmax[j], j == 0, lambda, mfinal);
                    out.block_exp[row * nb + j] = bp.bexp;
                }
                const int kindp = pack_kind<BPW>(bp.kind);
#pragma unroll
                for (int k = 0; k < NQ; ++k) {
                    const int src = k * BPW + lane / LPB;
                    const float mref = __shfl_sync(0xffffffffu, bp.mref, src);
                    const float be = __shfl_sync(0xffffffffu, bp.scale, src);
                const int kp = __shfl_sync(0xffffffffu, kindp, src);
                    const float4 x = qq < 2 ? v[qq * NQ + k] : piece[qq - 1][vi0 + k * THREADS];
                    dsum += emit_codes(c4 + qq * (kQuarter / 4) + vi0 + k * THREADS,
                                       block_words<true>(x, mref, (kp & 4) != 0, s_rep, s_lut, lane), be);
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, o);
            if (lane == 0) s_red[warp] = dsum;
            __syncthreads();                    // nobody reads the pieces (or the block arrays) any more
            if (tid == 0) {
                if (more) { request(1, row + gridDim.x, 2); request(2, row + gridDim.x, 3); }
                float t = 0.f;
#pragma unroll
                for (int i = 0; i < kWarps; ++i) t += s_red[i];
                out.row_d[row] = t;
            }
        } else {
            float4 *p4 = reinterpret_cast<float4 *>(out.probs + row * cols);
            BlockParams bp[4];
            int kindp[4];
#pragma unroll
            for (int qq = 0; qq < 4; ++qq) {
                bp[qq] = {0.f, 0.f, 1};
                if (lane < NQ * BPW) {
                    const int j = qq * nbq + jl;
                    bp[qq] = block_params(s_mbefore[j], s_bmax[j], j == 0, lambda, mfinal);
                }
                kindp[qq] = pack_kind<BPW>(bp[qq].kind);
            }
            auto weights = [&](int qq, int k, const float4 &x) {
                const int src = k * BPW + lane / LPB;
                const float mref = __shfl_sync(0xffffffffu, bp[qq].mref, src), scale = __shfl_sync(0xffffffffu, bp[qq].scale, src);
                const int kp = __shfl_sync(0xffffffffu, kindp[qq], src);
                return block_weights<true>(x, mref, scale, kp & 3, (kp & 4) != 0, f_rep, f_lut, lane);
            };
            // ---- weights of all four quarters (moved to the final max) and their sum -----------------------
#pragma unroll
            for (int qq = 0; qq < 2; ++qq)
#pragma unroll
                for (int k = 0; k < NQ; ++k) {
                    v[qq * NQ + k] = weights(qq, k, v[qq * NQ + k]);
                    dsum += (v[qq * NQ + k].x + v[qq * NQ + k].y) + (v[qq * NQ + k].z + v[qq * NQ + k].w);
                }
#pragma unroll
            for (int qq = 2; qq < 4; ++qq)
#pragma unroll
                for (int k = 0; k < NQ; ++k) {
                    const float4 w = weights(qq, k, piece[qq - 1][vi0 + k * THREADS]);
                    dsum += (w.x + w.y) + (w.z + w.w);
                }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, o);
            if (lane == 0) s_red[warp] = dsum;
            __syncthreads();
            float t = 0.f;                      // every thread adds the partial sums itself, in the same order
#pragma unroll
            for (int i = 0; i < kWarps; ++i) t += s_red[i];
            const float dinv = 1.f / t;
            // ---- output: quarters 0 and 1 from registers, 2 and 3 formed again from their pieces -----------
#pragma unroll
            for (int k = 0; k < 2 * NQ; ++k)
                __stcs(p4 + (k / NQ) * (kQuarter / 4) + vi0 + (k % NQ) * THREADS,
                       make_float4(v[k].x * dinv, v[k].y * dinv, v[k].z * dinv, v[k].w * dinv));
#pragma unroll
            for (int qq = 2; qq < 4; ++qq) {
#pragma unroll
                for (int k = 0; k < NQ; ++k) {
                    const float4 w = weights(qq, k, piece[qq - 1][vi0 + k * THREADS]);
                    __stcs(p4 + qq * (kQuarter / 4) + vi0 + k * THREADS, make_float4(w.x * dinv, w.y * dinv, w.z * dinv, w.w * dinv));
                }
                __syncthreads();                // nobody reads this piece any more (after the last one: nor the block arrays)
                if (tid == 0 && more) request(qq - 1, row + gridDim.x, qq);
            }
        }
    }
}

// Rows of up to 8K columns, several rows per CTA: GROUPS groups of THREADS threads each own one row
// at a time (register-resident, NV 16-byte vectors per thread; PF: the next row's loads always in flight,
// into a second set of registers) and share the CTA's tables; a group synchronises through its own
// hardware barrier (three per row), so the groups drift freely against each other.  With the tables
// shared, an SM holds as many rows in flight as its threads allow, where one-row CTAs stop at the six or
// seven copies of the 25 KB table that fit its shared memory.  CODES: 8-bit output.
template <int BK, int THREADS, int NV, int GROUPS, bool CODES, bool PF = true, bool REDUX = true>
__global__ void __launch_bounds__(THREADS * GROUPS)
softmax_rows_group_kernel(const float *__restrict__ logits, RowsOut out, int64_t rows, int lambda)
{
    constexpr int cols = NV * THREADS * 4, nb = cols / BK, kWarps = THREADS / 32;
    constexpr int LPB = BK / 4, BPW = 32 / LPB;
    static_assert(GROUPS >= 1 && GROUPS <= 15 && NV * BPW <= 32, "barrier ids 1 .. 15; one block per lane");
    __shared__ float s_bmax[GROUPS][nb];
    __shared__ float s_mbefore[GROUPS][nb];
    __shared__ uint32_t s_lut[kLutN];
    __shared__ __align__(16) uint32_t s_rep[(16 + kLutNegN) * 32];
    __shared__ float s_red[GROUPS][kWarps];
    __shared__ float s_mfinal[GROUPS];
    fill_tables<CODES, THREADS * GROUPS>(s_lut, s_rep, threadIdx.x);
    __syncthreads();
    const int grp = threadIdx.x / THREADS, tid = threadIdx.x % THREADS, lane = tid & 31, warp = tid >> 5;
    auto gsync = [&] {
        if (GROUPS == 1) __syncthreads();
        else asm volatile("bar.sync %0, %1;" ::"r"(1 + grp), "r"(THREADS) : "memory");
    };
    const int64_t stride = (int64_t)gridDim.x * GROUPS;
    int64_t row = (int64_t)blockIdx.x * GROUPS + grp;
    float4 vn[PF ? NV : 1];
    if (PF && row < rows) {
        const float4 *x4 = reinterpret_cast<const float4 *>(logits + row * cols);
#pragma unroll
        for (int k = 0; k < (PF ? NV : 1); ++k) vn[k] = __ldcs(x4 + (warp + k * kWarps) * 32 + lane);
    }
    for (; row < rows; row += stride) {
        float4 v[NV];
        if constexpr (PF) {
#pragma unroll
            for (int k = 0; k < NV; ++k) v[k] = vn[k];
            if (row + stride < rows) {
                const float4 *xn = reinterpret_cast<const float4 *>(logits + (row + stride) * cols);
#pragma unroll
                for (int k = 0; k < NV; ++k) vn[k] = __ldcs(xn + (warp + k * kWarps) * 32 + lane);
            }
        } else {
            const float4 *x4 = reinterpret_cast<const float4 *>(logits + row * cols);
#pragma unroll
            for (int k = 0; k < NV; ++k) v[k] = __ldcs(x4 + (warp + k * kWarps) * 32 + lane);
        }
        // ---- block maxima -------------------------------------------------------------------------
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            float mx = fmaxf(fmaxf(v[k].x, v[k].y), fmaxf(v[k].z, v[k].w));
            mx = lanes_max<LPB, REDUX>(mx);
            if ((lane % LPB) == 0) s_bmax[grp][(warp + k * kWarps) * BPW + lane / LPB] = mx;
        }
        gsync();
        // ---- scan over the blocks (the group's warp 0) ----------------------------------------------
        if (warp == 0) scan_blocks<nb>(s_bmax[grp], s_mbefore[grp], &s_mfinal[grp], lambda, lane);
        gsync();
        const float mfinal = s_mfinal[grp];
        const int jmine = (warp + (lane / BPW) * kWarps) * BPW + lane % BPW;      // the block whose parameters I work out
        float dsum = 0.f;
        if constexpr (CODES) {
            // ---- codes, block exponents, the sum of the decoded weights ------------------------------
            uint32_t *c4 = reinterpret_cast<uint32_t *>(out.codes + row * cols);
            CodesBlockParams bp = {0.f, 0, 1, 0.f};
            if (lane < NV * BPW) {
                bp = codes_block_params(s_mbefore[grp][jmine], s_bmax[grp][jmine], jmine == 0, lambda, mfinal);
                out.block_exp[row * nb + jmine] = bp.bexp;
            }
            const int kindp = pack_kind<BPW>(bp.kind);
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int src = k * BPW + lane / LPB;
                const float mref = __shfl_sync(0xffffffffu, bp.mref, src);
                const float be = __shfl_sync(0xffffffffu, bp.scale, src);
                const int kp = __shfl_sync(0xffffffffu, kindp, src);
                dsum += emit_codes(c4 + (warp + k * kWarps) * 32 + lane,
                                   block_words<true>(v[k], mref, (kp & 4) != 0, s_rep, s_lut, lane), be);
            }
        } else {
            // ---- weights (already moved to the final max) and their sum ------------------------------
            BlockParams bp = {0.f, 0.f, 1};
            if (lane < NV * BPW) bp = block_params(s_mbefore[grp][jmine], s_bmax[grp][jmine], jmine == 0, lambda, mfinal);
            const int kindp = pack_kind<BPW>(bp.kind);
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int src = k * BPW + lane / LPB;
                const float mref = __shfl_sync(0xffffffffu, bp.mref, src), scale = __shfl_sync(0xffffffffu, bp.scale, src);
                const int kp = __shfl_sync(0xffffffffu, kindp, src);
                v[k] = block_weights<true>(v[k], mref, scale, kp & 3, (kp & 4) != 0, reinterpret_cast<const float *>(s_rep),
                                           reinterpret_cast<const float *>(s_lut), lane);
                dsum += (v[k].x + v[k].y) + (v[k].z + v[k].w);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, o);
        if (lane == 0) s_red[grp][warp] = dsum;
        gsync();
        if constexpr (CODES) {
            if (tid == 0) {
                float t = 0.f;
#pragma unroll
                for (int i = 0; i < kWarps; ++i) t += s_red[grp][i];
                out.row_d[row] = t;
            }
        } else {
            // every thread adds the warps' partial sums itself, in the same order
            float t = 0.f;
#pragma unroll
            for (int i = 0; i < kWarps; ++i) t += s_red[grp][i];
            const float dinv = 1.f / t;
            float4 *p4 = reinterpret_cast<float4 *>(out.probs + row * cols);
#pragma unroll
            for (int k = 0; k < NV; ++k)
                __stcs(p4 + (warp + k * kWarps) * 32 + lane,
                       make_float4(v[k].x * dinv, v[k].y * dinv, v[k].z * dinv, v[k].w * dinv));
        }
        // (no barrier here: what the next row writes first, s_bmax, was last read before the third barrier
        // above; s_mfinal and s_red are written behind the next row's first and second barrier, which every
        // thread -- the one adding up s_red included -- joins only when it is done with this row)
    }
}

// Short rows (1K columns): one warp per row, the row in registers, no block-wide barrier at all.
// Lane l holds the float4 number l of every 128-element chunk; a block of Algorithm 1 is a whole
// chunk (BK = 128) or half of one (BK = 64).  Block maxima by a warp reduction, the scan replicated in
// every lane (it is a handful of scalar steps per block), weights, warp-wide sum, write.  CODES: 8-bit output.
template <int BK, int NV, bool CODES>
__global__ void __launch_bounds__(512)
softmax_rows_warp_kernel(const float *__restrict__ logits, RowsOut out, int64_t rows, int lambda)
{
    __shared__ uint32_t s_lut[kLutN];
    __shared__ __align__(16) uint32_t s_rep[(16 + kLutNegN) * 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int LPB = BK / 4, BPW = 32 / LPB, cols = NV * 128, nb = cols / BK;
    static_assert(NV * BPW <= 32, "one block per lane");
    fill_tables<CODES, 512>(s_lut, s_rep, tid);
    __syncthreads();
    const int myq = lane / LPB;                                  // which block of a chunk my lane is in
    const int64_t nwarps = (int64_t)gridDim.x * 16;
    for (int64_t row = (int64_t)blockIdx.x * 16 + warp; row < rows; row += nwarps) {
        const float4 *x4 = reinterpret_cast<const float4 *>(logits + row * cols);
        float4 v[NV];
        float bmx[NV];
#pragma unroll
        for (int k = 0; k < NV; ++k) v[k] = __ldcs(x4 + k * 32 + lane);
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            float mx = fmaxf(fmaxf(v[k].x, v[k].y), fmaxf(v[k].z, v[k].w));
            mx = lanes_max<LPB>(mx);
            bmx[k] = mx;                                         // maximum of my block of chunk k
        }
        // scan over the blocks in order, identical in every lane; lane BPW * k + q keeps what block q of
        // vector k saw (the max before it and its own maximum) and works out that block's parameters
        float m = -INFINITY, my_mb = -INFINITY, my_bm = -INFINITY;
#pragma unroll
        for (int k = 0; k < NV; ++k) {
#pragma unroll
            for (int q = 0; q < BPW; ++q) {
                const float bj = __shfl_sync(0xffffffffu, bmx[k], q * LPB);
                if (lane == k * BPW + q) { my_mb = m; my_bm = bj; }
                bool rs; float dl;
                m = row_block_update(m, bj, k == 0 && q == 0, lambda, &rs, &dl);
            }
        }
        const float mfinal = m;
        float dsum = 0.f;
        if constexpr (CODES) {
            uint32_t *c4 = reinterpret_cast<uint32_t *>(out.codes + row * cols);
            CodesBlockParams bp = {0.f, 0, 1, 0.f};
            if (lane < NV * BPW) {
                bp = codes_block_params(my_mb, my_bm, lane == 0, lambda, mfinal);
                out.block_exp[row * nb + lane] = bp.bexp;
            }
            const int kindp = pack_kind<BPW>(bp.kind);
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int src = k * BPW + myq;
                const float mref = __shfl_sync(0xffffffffu, bp.mref, src);
                const float be = __shfl_sync(0xffffffffu, bp.scale, src);
                const int kp = __shfl_sync(0xffffffffu, kindp, src);
                dsum += emit_codes(c4 + k * 32 + lane, block_words<true>(v[k], mref, (kp & 4) != 0, s_rep, s_lut, lane), be);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, o);
            if (lane == 0) out.row_d[row] = dsum;
        } else {
            float4 *p4 = reinterpret_cast<float4 *>(out.probs + row * cols);
            BlockParams bp = {0.f, 0.f, 1};
            if (lane < NV * BPW) bp = block_params(my_mb, my_bm, lane == 0, lambda, mfinal);
            const int kindp = pack_kind<BPW>(bp.kind);
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int src = k * BPW + myq;
                const float mref = __shfl_sync(0xffffffffu, bp.mref, src), scale = __shfl_sync(0xffffffffu, bp.scale, src);
                const int kp = __shfl_sync(0xffffffffu, kindp, src);
                v[k] = block_weights<true>(v[k], mref, scale, kp & 3, (kp & 4) != 0, reinterpret_cast<const float *>(s_rep),
                                           reinterpret_cast<const float *>(s_lut), lane);
                dsum += (v[k].x + v[k].y) + (v[k].z + v[k].w);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, o);
            const float dinv = 1.f / dsum;
#pragma unroll
            for (int k = 0; k < NV; ++k)
                __stcs(p4 + k * 32 + lane, make_float4(v[k].x * dinv, v[k].y * dinv, v[k].z * dinv, v[k].w * dinv));
        }
    }
}

// Row softmax with 8-bit output: the weights leave as HiF8 codes (Algorithm 1's "P in 8-bit") with one
// integer exponent per block and one denominator per row,
//     probs[r, c] = value(codes[r, c]) * 2^(block_exp[r, c / BK]) / row_d[r],
// 5 bytes of HBM traffic per element (4 in, 1 out) instead of 8.  Same max bookkeeping as above; block 0
// is not kept in high precision here (its weights take the 8-bit exponential like all others: the
// output has 8 bits anyway).  block_exp = (max the block's T were taken against) - (final max) <= 0.
// The table entries carry value and code in one word: a HiF8 value has at most four significant mantissa
// bits, so the low byte of its fp32 pattern is free for the code.  Blocks whose T are all <= 0 take their
// table word from a bank-replicated copy keyed by the top bits of -T * 2^-120 (as in the float-output
// kernels above).
// Any row length that is a multiple of 128: one CTA per row at a time; pass 1 block maxima (the HBM
// read), scan by warp 0, pass 2 re-reads the row (from L2), looks every T up and sums the decoded weights.
template <int BK, int THREADS, bool FAST>
__global__ void __launch_bounds__(THREADS)
softmax_rows_codes_generic_kernel(const float *__restrict__ logits, uint8_t *__restrict__ codes,
                                  int32_t *__restrict__ block_exp, float *__restrict__ row_d, int64_t rows, int cols,
                                  int lambda)
{
    __shared__ float s_bmax[kSrMaxBlocks];
    __shared__ float s_mbefore[kSrMaxBlocks];
    __shared__ uint32_t s_lut[kLutN];
    __shared__ __align__(16) uint32_t s_rep[FAST ? (16 + kLutNegN) * 32 : 32];
    __shared__ float s_red[THREADS / 32];
    __shared__ float s_mfinal;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int kWarps = THREADS / 32;
    constexpr int LPB = BK / 4, BPW = 32 / LPB;
    const int nb = cols / BK, nchunks = cols / 128;
    for (int i = tid; i < kLutN; i += THREADS) s_lut[i] = w0_word(g_w0_table[i]);
    for (int e = tid; FAST && e < 16 + kLutNegN; e += THREADS) {
        const uint32_t u = w0_word((e < 16) ? 1.f : g_w0_table[e - 16]);
        const uint4 u4 = make_uint4(u, u, u, u);
#pragma unroll
        for (int i = 0; i < 8; ++i) reinterpret_cast<uint4 *>(s_rep)[e * 8 + i] = u4;
    }
    __syncthreads();
    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const float4 *x4 = reinterpret_cast<const float4 *>(logits + row * cols);
        uint32_t *c4 = reinterpret_cast<uint32_t *>(codes + row * cols);
        for (int ch = warp; ch < nchunks; ch += kWarps) {
            const float4 x = __ldg(x4 + ch * 32 + lane);
            float mx = fmaxf(fmaxf(x.x, x.y), fmaxf(x.z, x.w));
            mx = lanes_max<LPB>(mx);
            if ((lane % LPB) == 0) s_bmax[ch * BPW + lane / LPB] = mx;
        }
        __syncthreads();
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
                    const bool pred = pending && fmaf(mj, kLog2e, -m) >= 1.1920928955078125e-07f;
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
        float dsum = 0.f;
        for (int ch = warp; ch < nchunks; ch += kWarps) {
            const float4 x = __ldg(x4 + ch * 32 + lane);
            const int j = ch * BPW + lane / LPB;
            const CodesBlockParams bp = codes_block_params(s_mbefore[j], s_bmax[j], j == 0, lambda, mfinal);
            // some lane of the warp holds a block with a positive T: voted by the whole warp
            const bool any_pos = __any_sync(0xffffffffu, bp.kind == 2);
            const uint4 e = block_words<FAST>(x, bp.mref, any_pos, s_rep, s_lut, lane);
            dsum += ((__uint_as_float(e.x & 0xFFFFFF00u) + __uint_as_float(e.y & 0xFFFFFF00u)) +
                     (__uint_as_float(e.z & 0xFFFFFF00u) + __uint_as_float(e.w & 0xFFFFFF00u))) * bp.scale;
            __stcs(c4 + ch * 32 + lane, (e.x & 0xFFu) | ((e.y & 0xFFu) << 8) | ((e.z & 0xFFu) << 16) | (e.w << 24));
            if ((lane % LPB) == 0) block_exp[row * nb + j] = bp.bexp;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, o);
        if (lane == 0) s_red[warp] = dsum;
        __syncthreads();
        if (tid == 0) {
            float t = 0.f;
            for (int i = 0; i < kWarps; ++i) t += s_red[i];
            row_d[row] = t;
        }
        __syncthreads();   // s_bmax / s_mbefore / s_red are reused by the next row
    }
}

template <int BK>
inline baps_status softmax_rows_codes_dispatch(const float *logits, uint8_t *codes, int32_t *block_exp, float *row_d,
                                               int64_t rows, int cols, int lambda, int num_sms, cudaStream_t st)
{
    const baps_status ts = ensure_w0_table(st);
    if (ts != BAPS_OK) return ts;
    auto grid_for = [&](int ctas_per_sm) {
        const int64_t cap = (int64_t)num_sms * ctas_per_sm;
        return (int)(rows < cap ? rows : cap);
    };
    // (grids as in the float-output dispatch below: several times what is resident)
    const RowsOut out = {nullptr, codes, block_exp, row_d};
    auto ring = [&](auto kernel, int threads, int dyn, int ctas_per_sm) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn) != cudaSuccess)
            return BAPS_ERR_CUDA;
        kernel<<<grid_for(ctas_per_sm), threads, dyn, st>>>(logits, out, rows, lambda);
        return BAPS_OK;
    };
    auto group = [&](auto kernel, int threads, int groups, int ctas) {
        const int64_t want = (rows + groups - 1) / groups, cap = (int64_t)num_sms * ctas;
        kernel<<<(int)(want < cap ? want : cap), threads * groups, 0, st>>>(logits, out, rows, lambda);
    };
    switch (cols) {
    case 1024: {
        const int64_t want = (rows + 15) / 16, cap = (int64_t)num_sms * 32;
        softmax_rows_warp_kernel<BK, 8, true><<<(int)(want < cap ? want : cap), 512, 0, st>>>(logits, out, rows, lambda);
        break;
    }
    case 2048:  group(softmax_rows_group_kernel<BK, 128, 4, 4, true, true>, 128, 4, 16); break;
    case 4096:  group(softmax_rows_group_kernel<BK, 256, 4, 4, true, true>, 256, 4, 4); break;
    case 8192:  group(softmax_rows_group_kernel<BK, 256, 8, 4, true, false>, 256, 4, 4); break;
    case 16384: if (ring(softmax_rows_ring_kernel<BK, 512, true>, 512, 65536, 2) != BAPS_OK) return BAPS_ERR_CUDA; break;
    case 32768: if (ring(softmax_rows_ring_kernel<BK, 1024, true>, 1024, 131072, 2) != BAPS_OK) return BAPS_ERR_CUDA; break;
    case 65536: if (ring(softmax_rows_quarters_kernel<BK, true>, 1024, 196608, 2) != BAPS_OK) return BAPS_ERR_CUDA; break;
    default:
        // other lengths re-read the row: large CTAs for long rows so that the re-read finds it in L2
        if (cols > 8192)
            softmax_rows_codes_generic_kernel<BK, 1024, true><<<grid_for(2), 1024, 0, st>>>(logits, codes, block_exp, row_d, rows, cols, lambda);
        else
            softmax_rows_codes_generic_kernel<BK, 256, false><<<grid_for(8), 256, 0, st>>>(logits, codes, block_exp, row_d, rows, cols, lambda);
        break;
    }
    return launch_status();
}

// Launch the variant for the row length (see the head of this file).
template <int BK>
inline baps_status softmax_rows_dispatch(const float *logits, float *probs, int64_t rows, int cols, int lambda,
                                  int num_sms, cudaStream_t st)
{
    const baps_status ts = ensure_w0_table(st);
    if (ts != BAPS_OK) return ts;
    auto grid_for = [&](int ctas_per_sm) {
        const int64_t cap = (int64_t)num_sms * ctas_per_sm;
        return (int)(rows < cap ? rows : cap);
    };
    const RowsOut out = {probs, nullptr, nullptr, nullptr};
    auto ring = [&](auto kernel, int threads, int dyn, int ctas_per_sm) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn) != cudaSuccess)
            return BAPS_ERR_CUDA;
        kernel<<<grid_for(ctas_per_sm), threads, dyn, st>>>(logits, out, rows, lambda);
        return BAPS_OK;
    };
    // Grids: several times the CTAs that are resident at once (a few rows per CTA), so that the hardware
    // scheduler evens out the SMs; measured on 2^28 logits, a grid of exactly the resident CTAs -- each
    // with a fixed share of the rows -- loses 5 to 10 % to the slowest SM.
    // Up to 8K columns the rows are register-resident and several rows share a CTA and its tables
    // (softmax_rows_group_kernel: 16 or 32 elements per thread); at 1K a warp per row needs no barrier at
    // all.  At 16K and 32K only one or two CTAs fit an SM, and the ring lets the next row's read overlap
    // the current row's passes.
    auto group = [&](auto kernel, int threads, int groups, int ctas) {
        const int64_t want = (rows + groups - 1) / groups, cap = (int64_t)num_sms * ctas;
        kernel<<<(int)(want < cap ? want : cap), threads * groups, 0, st>>>(logits, out, rows, lambda);
    };
    switch (cols) {
    case 1024: {
        const int64_t want = (rows + 15) / 16, cap = (int64_t)num_sms * 32;
        softmax_rows_warp_kernel<BK, 8, false><<<(int)(want < cap ? want : cap), 512, 0, st>>>(logits, out, rows, lambda);
        break;
    }
    case 2048: group(softmax_rows_group_kernel<BK, 128, 4, 4, false, true>, 128, 4, 16); break;
    case 4096: group(softmax_rows_group_kernel<BK, 256, 4, 4, false, true, false>, 256, 4, 4); break;
    case 8192: group(softmax_rows_group_kernel<BK, 256, 8, 4, false, false>, 256, 4, 4); break;
    case 16384: if (ring(softmax_rows_ring_kernel<BK, 512, false, false>, 512, 65536, 2) != BAPS_OK) return BAPS_ERR_CUDA; break;
    case 32768: if (ring(softmax_rows_ring_kernel<BK, 1024, false>, 1024, 131072, 2) != BAPS_OK) return BAPS_ERR_CUDA; break;
    case 65536: if (ring(softmax_rows_quarters_kernel<BK, false>, 1024, 196608, 2) != BAPS_OK) return BAPS_ERR_CUDA; break;
    default:
        if (cols >= 32768) {
            // long rows are re-read in passes 2 and 3: few enough CTAs that the rows in flight stay in L2
            softmax_rows_generic_kernel<BK, 1024, true><<<grid_for(2), 1024, 0, st>>>(logits, probs, rows, cols, lambda);
        } else {
            softmax_rows_generic_kernel<BK, 256, false><<<grid_for(8), 256, 0, st>>>(logits, probs, rows, cols, lambda);
        }
        break;
    }
    return launch_status();
}

} // namespace baps
