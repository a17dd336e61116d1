/*
 * baps.h -- C ABI of the BAPS CUDA library for NVIDIA B200 (sm_100a).
 *
 * BAPS ("block-aware precision rescaling") is a low-precision softmax workflow for attention:
 * inside a FlashAttention-style loop over key tiles, every score tile after the first is
 * taken relative to an integer running row maximum, rounded to the 8-bit HiF8 format,
 * exponentiated with 8-bit input and output, and accumulated with exact power-of-two
 * rescaling; a tile whose 8-bit entries exceed a threshold lambda is "restarted" against a
 * fresh high-precision maximum.  (Paper: Section 3 and Algorithm 1; 8-bit exponent:
 * Algorithm 2 in Appendix A.1.)
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller; nothing is retained after
 *     the call's work has finished on `stream`.  Pointers must be 16-byte aligned.
 *   - `stream` is a CUDA stream handle (cudaStream_t / CUstream); 0 is the default stream.
 *     Calls are asynchronous: the return value reports argument validation and launch
 *     errors only.  A device-side wait that ran out of time (the tensor-core kernel bounds
 *     every wait on a barrier) is reported by baps_poll_async_error().
 *   - No exceptions cross this boundary.  There is no CPU fallback: without a CUDA device
 *     every call returns BAPS_ERR_CUDA.
 *   - HiF8 here means: 1 sign bit, a prefix-coded "dot" field (11 / 10 / 01 / 001 / 0001 /
 *     0000) selecting 4 / 3 / 2 / 1 / 0 exponent bits or the denormal range, a sign-magnitude
 *     exponent with hidden leading one, and 1 / 2 / 3 / 3 / 3 mantissa bits; denormals are
 *     2^(m-23); 0x00 is zero, 0x80 NaN, 0x6F / 0xEF +-infinity.  Conversion rounds to the
 *     nearest value with ties to the larger magnitude; |x| >= 40960 gives infinity and
 *     |x| < 2^-23 gives 0x00.
 */
#ifndef BAPS_H_
#define BAPS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int baps_status;
enum {
    BAPS_OK = 0,
    BAPS_ERR_INVALID_ARG = -1, /* null pointer, non-positive size, H % Hkv != 0, ...          */
    BAPS_ERR_UNSUPPORTED = -2, /* a shape outside the supported set listed per entry point   */
    BAPS_ERR_ALIGNMENT = -3,   /* a pointer that is not 16-byte aligned                      */
    BAPS_ERR_CUDA = -4,        /* a CUDA runtime / driver call failed (launch, no device)    */
    BAPS_ERR_TIMEOUT = -5,     /* a bounded device-side wait expired (see poll below)        */
    BAPS_ERR_SCRATCH_LIMIT = -6 /* the problem needs more built-in scratch than the library has */
};

/* Which workflow the attention kernel runs. */
enum {
    BAPS_MODE_E2E_HIF8 = 0, /* Algorithm 1: first key tile in high precision, the rest 8-bit */
    BAPS_MODE_EXACT = 1,    /* Eq. (2): fp32 online softmax with a real-valued max ("Default"
                               setup of Section 4.1); used for error reporting              */
    BAPS_MODE_EXP2_HIF8 = 2 /* "Exp2 HiF8" setup of Section 4.1: Eq. (2) with a real-valued max in
                               which every power of two -- the weights 2^(S - m) and the rescale
                               factor 2^(m_prev - m) -- takes an 8-bit HiF8 argument and gives an
                               8-bit HiF8 result (Algorithm 2); no restart, lambda is ignored */
};

enum { BAPS_DTYPE_BF16 = 0, BAPS_DTYPE_F32 = 1 };

typedef struct CUstream_st *baps_stream;

/* ---- HiF8 conversions (the conversions of Algorithm 2, lines "convert to HiF8" / "convert
 *      back") -------------------------------------------------------------------------------
 * encode: codes[i] = HiF8(x[i]); decode: x[i] = value(codes[i]) (NaN for 0x80).
 * x: n floats, codes: n bytes, both device memory.  n == 0 is a no-op returning BAPS_OK.   */
baps_status baps_hif8_encode(const float *x, uint8_t *codes, size_t n, baps_stream stream);
baps_status baps_hif8_decode(const uint8_t *codes, float *x, size_t n, baps_stream stream);

/* ---- 8-bit exponent (Algorithm 2; line "P = 2^T, in 8-bit" of Algorithm 1) ------------------
 * p_codes[i] = HiF8(2^value(t_codes[i])): 8-bit in, 8-bit out.  NaN -> NaN, -Inf -> 0,
 * overflow -> +Inf.  Device pointers, n bytes each.                                          */
baps_status baps_exp2_hif8(const uint8_t *t_codes, uint8_t *p_codes, size_t n, baps_stream stream);

/* ---- Row softmax by Algorithm 1 restricted to single rows (the non-fused path) ---------------
 * logits, probs: [rows, cols] float32 row-major, device memory.  logits are natural-log
 * logits: the base-2 score is s = logit * log2(e).  The row is cut into blocks of block_k
 * entries; block 0 is the high-precision tile (set B0), every later block is rounded to HiF8
 * relative to the integer running maximum, with a per-row restart at lambda = 1.
 * probs[r, c] = w[r, c] * 2^(m_block(c) - m_final) / d.
 * Supported: block_k in {64, 128}, cols % 128 == 0 (the kernels walk the row in 128-element warp
 * steps, also when block_k is 64), cols <= 65536 (BAPS_ERR_UNSUPPORTED otherwise); rows == 0 is a
 * no-op.                                                                                      */
baps_status baps_softmax_rows(const float *logits, float *probs, int64_t rows, int64_t cols,
                              int block_k, baps_stream stream);

/* ---- Row softmax with 8-bit output (Algorithm 1, line "P = 2^T, in 8-bit": the weights are 8-bit
 *      numbers; this entry point hands them out as such) ----------------------------------------
 * Same row-wise workflow as baps_softmax_rows, but the result leaves as
 *     probs[r, c] = value(codes[r, c]) * 2^(block_exp[r, c / block_k]) / row_d[r]
 * with codes: [rows, cols] HiF8 codes, block_exp: [rows, cols / block_k] int32 (<= 0: the max the
 * block's T were taken against minus the final max) and row_d: [rows] float32 -- 5 bytes of memory
 * traffic per element instead of 8.  Block 0 is not a high-precision tile in this variant: its
 * weights take the 8-bit exponential like all others; its maximum still initialises the integer
 * max.  T is formed in single precision with one rounding, T = fl(x * fl(log2 e) - m).
 * All pointers are device memory; logits and codes 16-byte aligned, block_exp and row_d 4-byte.
 * Supported set as for baps_softmax_rows.                                                       */
baps_status baps_softmax_rows_codes(const float *logits, uint8_t *codes, int32_t *block_exp, float *row_d,
                                    int64_t rows, int64_t cols, int block_k, baps_stream stream);

/* ---- Fused attention forward (Algorithm 1 around the tiling of Eq. (2)) ----------------------
 * q, out: [B, H, S, D]; k, v: [B, Hkv, S, D]; contiguous, D innermost, bfloat16.  Query head h
 * reads kv head h / (H / Hkv).  Scale 1/sqrt(D), lambda = 1, B0 = the first key tile.
 * causal != 0 masks keys c > r (masked scores are -inf; fully masked tiles are skipped).
 * Results depend on block_q and block_k by design: the restart decision is taken per
 * block_q x block_k tile.
 * Supported (else BAPS_ERR_UNSUPPORTED): D in {64, 128}; H % Hkv == 0;
 * (block_q, block_k) = (128, 128); S % 128 == 0.                                             */
baps_status baps_attention_fwd(const void *q, const void *k, const void *v, void *out,
                               int B, int H, int Hkv, int S, int D, int causal,
                               int block_q, int block_k, baps_stream stream);

/* Same problem with float32 inputs and output; scores are accumulated in double precision on
 * the CUDA cores (a slow, small-problem path; the configuration with S = 128, D = 64, 64 x 64
 * tiles uses it).  Supported: D <= 128 and D % 4 == 0; (block_q, block_k) in {(64, 64),
 * (128, 128)}; S % block_q == 0.                                                             */
baps_status baps_attention_fwd_f32(const float *q, const float *k, const float *v, float *out,
                                   int B, int H, int Hkv, int S, int D, int causal,
                                   int block_q, int block_k, baps_stream stream);

/* Options and optional instrumentation of the extended call.  Every pointer of baps_stats may
 * be NULL; the non-NULL ones are device buffers the kernel fills. */
typedef struct {
    int lambda;  /* restart threshold, integer (Section 4.4), 0..3; Algorithm 1 default 1;
                    ignored by the modes that have no restart                                 */
    int mode;    /* BAPS_MODE_*                                                               */
    float scale; /* softmax scale; 0 selects 1/sqrt(D)                                        */
    int b0_last; /* 0: the high-precision set B0 is the first key tile (Section 4.1's setup);
                    non-zero: B0 = {first, last visible key tile} -- Section 3.2 notes that in
                    causal language models the first and the last tile usually hold the large
                    scores.  The key tiles are then visited in the order 0, last, 1, ..., last - 1
                    (last = the diagonal tile when causal), the first two in high precision.
                    Algorithm 1 only; the tensor-core kernel then runs one query tile per CTA.     */
} baps_opts;

/* out_f32 must be 16-byte aligned, the others 4-byte aligned (BAPS_ERR_ALIGNMENT otherwise). */
typedef struct {
    float *row_m;      /* [B, H, S] final integer running maximum m                          */
    float *row_d;      /* [B, H, S] final denominator d                                      */
    int32_t *restarts; /* [B, H, S / block_q] number of restarted tiles (Table 4's counter)  */
    float *out_f32;    /* [B, H, S, D] output before rounding to the storage type            */
} baps_stats;

/* dtype: BAPS_DTYPE_BF16 selects the tensor-core kernel (same supported set as
 * baps_attention_fwd), BAPS_DTYPE_F32 the CUDA-core kernel.  `out` may be NULL if
 * stats->out_f32 is given.  opts == NULL means {1, BAPS_MODE_E2E_HIF8, 0, 0}.               */
baps_status baps_attention_fwd_ex(const void *q, const void *k, const void *v, void *out,
                                  int B, int H, int Hkv, int S, int D, int causal,
                                  int block_q, int block_k, int dtype, const baps_opts *opts,
                                  const baps_stats *stats, baps_stream stream);

/* ---- Quantised Q and K (Section 3.4: "can be fused with the dequantization step when Q_i and K_j are
 *      hardware-quantized"; also the outlook of the conclusion) -------------------------------------
 * q8: [B, H, S, D], k8: [B, Hkv, S, D] FP8 E4M3 codes (OCP, bias 7), one byte per element;
 * q_scale: [B, H, S / 128], k_scale: [B, Hkv, S / 128] float32 dequantisation scales, one per 128-row
 * tile, which must be powers of two: element (r, t) of Q stands for value(q8[r, t]) * q_scale[r / 128].
 * v, out: bfloat16 as in baps_attention_fwd.  Q K^T runs on the 8-bit tensor-core path with FP32
 * accumulation (exact products), and the two scales of a tile pair are folded into the score scale,
 * so that S = (Q8 K8^T) * (q_scale * k_scale * log2(e) * scale) -- everything after that is
 * Algorithm 1 (or the mode opts selects) unchanged.  opts and stats as in baps_attention_fwd_ex;
 * either may be NULL.  Supported: D = 128, (block_q, block_k) = (128, 128), S % 128 == 0.          */
baps_status baps_attention_fwd_fp8(const uint8_t *q8, const uint8_t *k8, const void *v, void *out,
                                   const float *q_scale, const float *k_scale,
                                   int B, int H, int Hkv, int S, int D, int causal,
                                   int block_q, int block_k, const baps_opts *opts,
                                   const baps_stats *stats, baps_stream stream);

/* ---- Restart-rate statistics (Section 4.4, Table 4) ---------------------------------------------
 * Runs the fused attention exactly as baps_attention_fwd_ex(dtype bf16, mode E2E_HIF8, given
 * lambda) does -- `out` receives the attention output -- while counting, per query tile, the
 * 8-bit key tiles that had to be restarted, and reduces the counts to
 *   rates[0] = ARR, restarted tiles / 8-bit tiles over the whole call, and
 *   rates[1] = PRR, the largest such ratio over the query tiles ("any single calculation of O_i").
 * scratch: device int32 buffer of at least B * H * S / 128 entries owned by the caller; it holds
 * the per-query-tile counters between the two kernels and its contents are overwritten.
 * scratch_entries: capacity of that buffer (BAPS_ERR_INVALID_ARG if too small).
 * rates: device float[2]; NaN, NaN if a device-side wait of this call expired (see
 * baps_poll_async_error).  Same supported set as baps_attention_fwd; lambda in 0..3.           */
baps_status baps_attention_restart_rates(const void *q, const void *k, const void *v, void *out,
                                         int B, int H, int Hkv, int S, int D, int causal,
                                         int block_q, int block_k, int lambda, int32_t *scratch,
                                         size_t scratch_entries, float *rates, baps_stream stream);

/* ---- Restart rates for callers that cannot allocate (no counterpart in the paper) ------------------
 * Same computation and same results as baps_attention_restart_rates, but the per-query-tile
 * counters live in a scratch array that is part of the library image instead of a buffer the
 * caller provides.  It is meant for callers that have no way to obtain device memory of their
 * own at the point of the call: code that runs under a host application which hands it a fixed
 * set of buffers and forbids further allocation, serving loops in which an allocation (which
 * may synchronise the whole device) is not acceptable, or processes in which another framework
 * owns the allocator.  The entry point itself never calls cudaMalloc, cudaFree or any routine
 * that allocates.
 *   - Limit: B * H * S / 128 <= BAPS_STATIC_SCRATCH_ENTRIES (262144 counters, 1 MiB per GPU that
 *     loads the library, held until the process exits).  Larger problems are refused with
 *     BAPS_ERR_SCRATCH_LIMIT; nothing is launched in that case.
 *   - The first call on a device looks up the device address of the array and, like the other
 *     attention entry points, builds the weight table; that first call synchronises the stream
 *     and should be made before any stream capture is started.
 *   - All calls on a device share the one array.  Every counter the reduction reads is rewritten
 *     by the attention kernel of the same call, so nothing has to be cleared between calls, but two
 *     calls whose kernels overlap on the GPU (different streams) race on it: serialise them.
 *   - Like every attention entry point the call returns before the kernels have run: `out` and
 *     `rates` are meaningful only if baps_poll_async_error() afterwards returns BAPS_OK.  After an
 *     expired device-side wait the counters of that call are incomplete and rates[0..1] are NaN.
 * q, k, v, out, rates and the remaining arguments are exactly those of
 * baps_attention_restart_rates.                                                               */
#define BAPS_STATIC_SCRATCH_ENTRIES 262144
baps_status baps_attention_restart_rates_static(const void *q, const void *k, const void *v, void *out,
                                                int B, int H, int Hkv, int S, int D, int causal,
                                                int block_q, int block_k, int lambda, float *rates,
                                                baps_stream stream);

/* Human-readable name of a status code (static string, never NULL). */
const char *baps_status_string(baps_status status);

/* Synchronises `stream`, then returns BAPS_ERR_TIMEOUT if any kernel launched by this library
 * on the current device has recorded an expired wait since the last poll (and clears the
 * record), BAPS_ERR_CUDA if the stream reports an error, else BAPS_OK. */
baps_status baps_poll_async_error(baps_stream stream);

/* Number of kernels this library has launched since it was loaded (for launch accounting). */
int64_t baps_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* BAPS_H_ */
