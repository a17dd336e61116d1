// C-ABI entry points of the BAPS CUDA library (declared in include/baps.h).
// One translation unit: the kernels live in the .cuh files included below.
#include "baps_common.cuh"
#include "baps_hif8.cuh"
#include "baps_elementwise.cuh"
#include "baps_softmax_rows.cuh"
#include "baps_attention_f32.cuh"
#include "baps_attention_tc.cuh"

#include <cmath>
#include <mutex>

using namespace baps;

namespace {

int num_sms()
{
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

template <typename K>
baps_status set_smem(K kernel, size_t bytes)
{
    if (bytes > 48 * 1024) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) !=
            cudaSuccess)
            return BAPS_ERR_CUDA;
    }
    return BAPS_OK;
}

baps_status attention_f32_launch(const AttnF32Params &p, int bq, int bk, cudaStream_t st)
{
    dim3 grid(p.S / bq, p.H, p.B);
    if (bq == 64) {
        const size_t sm = attention_f32_smem<64, 64>();
        if (set_smem(attention_f32_kernel<64, 64>, sm) != BAPS_OK) return BAPS_ERR_CUDA;
        attention_f32_kernel<64, 64><<<grid, kAfThreads, sm, st>>>(p);
    } else {
        const size_t sm = attention_f32_smem<128, 128>();
        if (set_smem(attention_f32_kernel<128, 128>, sm) != BAPS_OK) return BAPS_ERR_CUDA;
        attention_f32_kernel<128, 128><<<grid, kAfThreads, sm, st>>>(p);
    }
    return launch_status();
}

baps_status check_attention_common(const void *q, const void *k, const void *v, int B, int H,
                                   int Hkv, int S, int D)
{
    if (!q || !k || !v) return BAPS_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || Hkv <= 0 || S <= 0 || D <= 0) return BAPS_ERR_INVALID_ARG;
    if (H % Hkv != 0) return BAPS_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v)) return BAPS_ERR_ALIGNMENT;
    return BAPS_OK;
}

// Reduction of per-query-tile restart counters to the two rates of Table 4 (one CTA).
// Query tile i of a causal problem has i 8-bit key tiles (its first tile is the B0 tile), of a
// non-causal one nk - 1.
__global__ void __launch_bounds__(1024)
restart_rates_kernel(const int32_t *__restrict__ counts, int64_t n, int nq, int nk, int causal,
                     float *__restrict__ rates)
{
    __shared__ float s_r[32], s_t[32], s_p[32];
    float r = 0.f, tiles = 0.f, peak = 0.f;
    for (int64_t i = threadIdx.x; i < n; i += blockDim.x) {
        const int b1 = causal ? (int)(i % nq) : nk - 1;
        const float c = (float)counts[i];
        r += c; tiles += (float)b1;
        if (b1 > 0) peak = fmaxf(peak, c / (float)b1);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        r += __shfl_xor_sync(0xffffffffu, r, o);
        tiles += __shfl_xor_sync(0xffffffffu, tiles, o);
        peak = fmaxf(peak, __shfl_xor_sync(0xffffffffu, peak, o));
    }
    if ((threadIdx.x & 31) == 0) { s_r[threadIdx.x >> 5] = r; s_t[threadIdx.x >> 5] = tiles; s_p[threadIdx.x >> 5] = peak; }
    __syncthreads();
    if (threadIdx.x == 0) {
        float R = 0.f, T = 0.f, P = 0.f;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { R += s_r[w]; T += s_t[w]; P = fmaxf(P, s_p[w]); }
        // After an expired wait the attention kernel has not rewritten every counter: the rates
        // would mix in whatever the buffer held before, so they are reported as NaN instead.
        const bool failed = *reinterpret_cast<volatile int *>(&g_async_status) != 0;
        rates[0] = failed ? __int_as_float(0x7fc00000) : (T > 0.f ? R / T : 0.f);
        rates[1] = failed ? __int_as_float(0x7fc00000) : P;
    }
}

baps_status restart_rates_impl(const void *q, const void *k, const void *v, void *out, int B, int H, int Hkv,
                               int S, int D, int causal, int block_q, int block_k, int lambda,
                               int32_t *counts, float *rates, baps_stream stream)
{
    baps_opts o = {lambda, BAPS_MODE_E2E_HIF8, 0.f, 0};
    baps_stats st = {nullptr, nullptr, counts, nullptr};
    baps_status rc = baps_attention_fwd_ex(q, k, v, out, B, H, Hkv, S, D, causal, block_q, block_k,
                                           BAPS_DTYPE_BF16, &o, &st, stream);
    if (rc != BAPS_OK) return rc;
    const int nq = S / 128;
    restart_rates_kernel<<<1, 1024, 0, as_stream(stream)>>>(counts, (int64_t)B * H * nq, nq, nq, causal ? 1 : 0, rates);
    return launch_status();
}

// Built-in scratch of baps_attention_restart_rates_static: per-query-tile restart counters.
// In host code this name is only a stand-in for the symbol, not a device address; the address the
// kernels need is looked up once per device with cudaGetSymbolAddress (static_scratch_ptr below).
static __device__ __align__(256) int32_t g_static_restart_counts[BAPS_STATIC_SCRATCH_ENTRIES];

// Device address of the built-in scratch for the current device (looked up on first use with
// that device current); nullptr if the lookup fails.
int32_t *static_scratch_ptr()
{
    static int32_t *ptrs[64] = {nullptr};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> setup_lock(g_setup_mutex);
    if (!ptrs[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_restart_counts) != cudaSuccess) return nullptr;
        ptrs[dev] = static_cast<int32_t *>(p);
    }
    return ptrs[dev];
}

} // namespace

extern "C" {

const char *baps_status_string(baps_status s)
{
    switch (s) {
    case BAPS_OK: return "BAPS_OK";
    case BAPS_ERR_INVALID_ARG: return "BAPS_ERR_INVALID_ARG";
    case BAPS_ERR_UNSUPPORTED: return "BAPS_ERR_UNSUPPORTED";
    case BAPS_ERR_ALIGNMENT: return "BAPS_ERR_ALIGNMENT";
    case BAPS_ERR_CUDA: return "BAPS_ERR_CUDA";
    case BAPS_ERR_TIMEOUT: return "BAPS_ERR_TIMEOUT";
    case BAPS_ERR_SCRATCH_LIMIT: return "BAPS_ERR_SCRATCH_LIMIT (problem exceeds the built-in scratch)";
    default: return "BAPS_ERR_UNKNOWN";
    }
}

int64_t baps_launch_count(void) { return g_launches.load(); }

#ifdef BAPS_TEST_SKIP_LOAD
// Test build only: make the attention kernel's TMA producer leave out K / V tile load number l
// (0 = K_0, 1 = V_0, 2 = K_1, ...) in the launches that follow; -1 switches it off.
int baps_test_skip_kv_load(int l)
{
    return cudaMemcpyToSymbol(g_test_skip_load, &l, sizeof(int)) == cudaSuccess ? 0 : -1;
}
#endif

baps_status baps_poll_async_error(baps_stream stream)
{
    if (!have_device()) return BAPS_ERR_CUDA;
    cudaStream_t st = as_stream(stream);
    if (cudaStreamSynchronize(st) != cudaSuccess) return BAPS_ERR_CUDA;
    int host = 0;
    if (cudaMemcpyFromSymbol(&host, g_async_status, sizeof(int)) != cudaSuccess) return BAPS_ERR_CUDA;
    if (host != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_async_status, &zero, sizeof(int)) != cudaSuccess) return BAPS_ERR_CUDA;
        return BAPS_ERR_TIMEOUT;
    }
    return BAPS_OK;
}

// First call on a device: build the 8192-entry code table and the 256-entry exponent map and wait for
// them (later calls may come on any stream).
static baps_status ensure_ew_tables(cudaStream_t stream)
{
    static bool ready[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BAPS_ERR_CUDA;
    std::lock_guard<std::mutex> setup_lock(g_setup_mutex);
    if (!ready[dev]) {
        encode_table_init_kernel<<<8, 256, 0, stream>>>();
        if (cudaGetLastError() != cudaSuccess) return BAPS_ERR_CUDA;
        ++g_launches;
        if (cudaStreamSynchronize(stream) != cudaSuccess) return BAPS_ERR_CUDA;
        ready[dev] = true;
    }
    return BAPS_OK;
}

baps_status baps_hif8_encode(const float *x, uint8_t *codes, size_t n, baps_stream stream)
{
    if (n == 0) return BAPS_OK;
    if (!x || !codes) return BAPS_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(codes)) return BAPS_ERR_ALIGNMENT;
    if (!have_device()) return BAPS_ERR_CUDA;
    const baps_status ts = ensure_ew_tables(as_stream(stream));
    if (ts != BAPS_OK) return ts;
    const size_t units = n / 4 / ((size_t)kEwThreads * kEwUnroll);
    hif8_encode_kernel<<<ew_grid(units, num_sms()), kEwThreads, 0, as_stream(stream)>>>(x, codes, n);
    return launch_status();
}

baps_status baps_hif8_decode(const uint8_t *codes, float *x, size_t n, baps_stream stream)
{
    if (n == 0) return BAPS_OK;
    if (!x || !codes) return BAPS_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(codes)) return BAPS_ERR_ALIGNMENT;
    if (!have_device()) return BAPS_ERR_CUDA;
    const size_t units = n / 16 / (size_t)kEwThreads;
    hif8_decode_kernel<<<ew_grid(units, num_sms()), kEwThreads, 0, as_stream(stream)>>>(codes, x, n);
    return launch_status();
}

baps_status baps_exp2_hif8(const uint8_t *t_codes, uint8_t *p_codes, size_t n, baps_stream stream)
{
    if (n == 0) return BAPS_OK;
    if (!t_codes || !p_codes) return BAPS_ERR_INVALID_ARG;
    if (!aligned16(t_codes) || !aligned16(p_codes)) return BAPS_ERR_ALIGNMENT;
    if (!have_device()) return BAPS_ERR_CUDA;
    const baps_status ts = ensure_ew_tables(as_stream(stream));
    if (ts != BAPS_OK) return ts;
    const size_t units = n / 16 / ((size_t)kEwThreads * 2);
    hif8_exp2_kernel<<<ew_grid(units, num_sms(), 8), kEwThreads, 0, as_stream(stream)>>>(t_codes, p_codes, n);
    return launch_status();
}

baps_status baps_softmax_rows(const float *logits, float *probs, int64_t rows, int64_t cols,
                              int block_k, baps_stream stream)
{
    if (rows < 0 || cols <= 0) return BAPS_ERR_INVALID_ARG;
    if (rows == 0) return BAPS_OK;
    if (!logits || !probs) return BAPS_ERR_INVALID_ARG;
    if ((block_k != 64 && block_k != 128) || cols % 128 != 0 || cols > 65536)
        return BAPS_ERR_UNSUPPORTED;
    if (!aligned16(logits) || !aligned16(probs)) return BAPS_ERR_ALIGNMENT;
    if (!have_device()) return BAPS_ERR_CUDA;
    if (block_k == 64)
        return softmax_rows_dispatch<64>(logits, probs, rows, (int)cols, 1, num_sms(), as_stream(stream));
    return softmax_rows_dispatch<128>(logits, probs, rows, (int)cols, 1, num_sms(), as_stream(stream));
}

baps_status baps_softmax_rows_codes(const float *logits, uint8_t *codes, int32_t *block_exp, float *row_d,
                                    int64_t rows, int64_t cols, int block_k, baps_stream stream)
{
    if (rows < 0 || cols <= 0) return BAPS_ERR_INVALID_ARG;
    if (rows == 0) return BAPS_OK;
    if (!logits || !codes || !block_exp || !row_d) return BAPS_ERR_INVALID_ARG;
    if ((block_k != 64 && block_k != 128) || cols % 128 != 0 || cols > 65536) return BAPS_ERR_UNSUPPORTED;
    if (!aligned16(logits) || !aligned16(codes) || !aligned4(block_exp) || !aligned4(row_d)) return BAPS_ERR_ALIGNMENT;
    if (!have_device()) return BAPS_ERR_CUDA;
    if (block_k == 64)
        return softmax_rows_codes_dispatch<64>(logits, codes, block_exp, row_d, rows, (int)cols, 1, num_sms(), as_stream(stream));
    return softmax_rows_codes_dispatch<128>(logits, codes, block_exp, row_d, rows, (int)cols, 1, num_sms(), as_stream(stream));
}

baps_status baps_attention_fwd_ex(const void *q, const void *k, const void *v, void *out,
                                  int B, int H, int Hkv, int S, int D, int causal,
                                  int block_q, int block_k, int dtype, const baps_opts *opts,
                                  const baps_stats *stats, baps_stream stream)
{
    baps_status st = check_attention_common(q, k, v, B, H, Hkv, S, D);
    if (st != BAPS_OK) return st;
    baps_opts o = {1, BAPS_MODE_E2E_HIF8, 0.f, 0};
    if (opts) o = *opts;
    baps_stats s = {nullptr, nullptr, nullptr, nullptr};
    if (stats) s = *stats;
    if (!out && !s.out_f32) return BAPS_ERR_INVALID_ARG;
    if (out && !aligned16(out)) return BAPS_ERR_ALIGNMENT;
    if (s.out_f32 && !aligned16(s.out_f32)) return BAPS_ERR_ALIGNMENT;      // written with 16-byte stores
    if (!aligned4(s.row_m) || !aligned4(s.row_d) || !aligned4(s.restarts)) return BAPS_ERR_ALIGNMENT;
    if (o.lambda < 0 || o.lambda > 3) return BAPS_ERR_UNSUPPORTED;
    if (o.mode != BAPS_MODE_E2E_HIF8 && o.mode != BAPS_MODE_EXACT && o.mode != BAPS_MODE_EXP2_HIF8)
        return BAPS_ERR_UNSUPPORTED;
    if (!(o.scale >= 0.f)) return BAPS_ERR_INVALID_ARG;
    const double scale = o.scale > 0.f ? (double)o.scale : 1.0 / std::sqrt((double)D);
    const double c = 1.4426950408889634074 * scale;

    if (dtype == BAPS_DTYPE_F32) {
        if (!((block_q == 64 && block_k == 64) || (block_q == 128 && block_k == 128)))
            return BAPS_ERR_UNSUPPORTED;
        if (D > 128 || D % 4 != 0 || S % block_q != 0) return BAPS_ERR_UNSUPPORTED;
        if (!have_device()) return BAPS_ERR_CUDA;
        AttnF32Params p;
        p.q = (const float *)q; p.k = (const float *)k; p.v = (const float *)v;
        p.out = (float *)out; p.row_m = s.row_m; p.row_d = s.row_d; p.out_f32 = s.out_f32;
        p.restarts = s.restarts;
        p.B = B; p.H = H; p.Hkv = Hkv; p.S = S; p.D = D; p.causal = causal ? 1 : 0;
        p.lambda = o.lambda; p.mode = o.mode; p.c = c; p.b0_last = o.b0_last ? 1 : 0;
        return attention_f32_launch(p, block_q, block_k, as_stream(stream));
    }
    if (dtype == BAPS_DTYPE_BF16) {
        if (block_q != 128 || block_k != 128) return BAPS_ERR_UNSUPPORTED;
        if (c < 0.03125 || c > 1024.0) return BAPS_ERR_UNSUPPORTED;   // log2(e) * scale window
        if ((D != 64 && D != 128) || S % 128 != 0) return BAPS_ERR_UNSUPPORTED;
        if ((long long)B * H * S > 0x7fffffffLL) return BAPS_ERR_UNSUPPORTED;   // 32-bit TMA row coordinate
        if (!have_device()) return BAPS_ERR_CUDA;
        return attention_tc_launch(q, k, v, out, B, H, Hkv, S, D, causal ? 1 : 0, o.lambda, o.mode,
                                   o.b0_last ? 1 : 0, (float)c, s, num_sms(), as_stream(stream));
    }
    return BAPS_ERR_INVALID_ARG;
}

baps_status baps_attention_fwd_fp8(const uint8_t *q8, const uint8_t *k8, const void *v, void *out,
                                   const float *q_scale, const float *k_scale,
                                   int B, int H, int Hkv, int S, int D, int causal,
                                   int block_q, int block_k, const baps_opts *opts,
                                   const baps_stats *stats, baps_stream stream)
{
    baps_status st = check_attention_common(q8, k8, v, B, H, Hkv, S, D);
    if (st != BAPS_OK) return st;
    if (!q_scale || !k_scale) return BAPS_ERR_INVALID_ARG;
    if (!aligned4(q_scale) || !aligned4(k_scale)) return BAPS_ERR_ALIGNMENT;
    baps_opts o = {1, BAPS_MODE_E2E_HIF8, 0.f, 0};
    if (opts) o = *opts;
    baps_stats s = {nullptr, nullptr, nullptr, nullptr};
    if (stats) s = *stats;
    if (!out && !s.out_f32) return BAPS_ERR_INVALID_ARG;
    if (out && !aligned16(out)) return BAPS_ERR_ALIGNMENT;
    if (s.out_f32 && !aligned16(s.out_f32)) return BAPS_ERR_ALIGNMENT;
    if (!aligned4(s.row_m) || !aligned4(s.row_d) || !aligned4(s.restarts)) return BAPS_ERR_ALIGNMENT;
    if (o.lambda < 0 || o.lambda > 3) return BAPS_ERR_UNSUPPORTED;
    if (o.mode != BAPS_MODE_E2E_HIF8 && o.mode != BAPS_MODE_EXACT && o.mode != BAPS_MODE_EXP2_HIF8)
        return BAPS_ERR_UNSUPPORTED;
    if (!(o.scale >= 0.f)) return BAPS_ERR_INVALID_ARG;
    if (block_q != 128 || block_k != 128 || D != 128 || S % 128 != 0) return BAPS_ERR_UNSUPPORTED;
    if ((long long)B * H * S > 0x7fffffffLL) return BAPS_ERR_UNSUPPORTED;
    const double scale = o.scale > 0.f ? (double)o.scale : 1.0 / std::sqrt((double)D);
    const double c = 1.4426950408889634074 * scale;
    if (!have_device()) return BAPS_ERR_CUDA;
    return attention_tc_launch(q8, k8, v, out, B, H, Hkv, S, D, causal ? 1 : 0, o.lambda, o.mode,
                               o.b0_last ? 1 : 0, (float)c, s, num_sms(), as_stream(stream), q_scale, k_scale);
}

baps_status baps_attention_restart_rates(const void *q, const void *k, const void *v, void *out,
                                         int B, int H, int Hkv, int S, int D, int causal,
                                         int block_q, int block_k, int lambda, int32_t *scratch,
                                         size_t scratch_entries, float *rates, baps_stream stream)
{
    if (!out || !scratch || !rates) return BAPS_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || S <= 0) return BAPS_ERR_INVALID_ARG;
    if (scratch_entries < (size_t)B * (size_t)H * (size_t)(S / 128)) return BAPS_ERR_INVALID_ARG;
    return restart_rates_impl(q, k, v, out, B, H, Hkv, S, D, causal, block_q, block_k, lambda, scratch, rates,
                              stream);
}

baps_status baps_attention_restart_rates_static(const void *q, const void *k, const void *v, void *out,
                                                int B, int H, int Hkv, int S, int D, int causal,
                                                int block_q, int block_k, int lambda, float *rates,
                                                baps_stream stream)
{
    if (!out || !rates) return BAPS_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || S <= 0) return BAPS_ERR_INVALID_ARG;
    if ((size_t)B * (size_t)H * (size_t)(S / 128) > (size_t)BAPS_STATIC_SCRATCH_ENTRIES)
        return BAPS_ERR_SCRATCH_LIMIT;
    if (!have_device()) return BAPS_ERR_CUDA;
    int32_t *counts = static_scratch_ptr();      // first call on this device: symbol address lookup
    if (!counts) return BAPS_ERR_CUDA;
    return restart_rates_impl(q, k, v, out, B, H, Hkv, S, D, causal, block_q, block_k, lambda, counts, rates,
                              stream);
}

baps_status baps_attention_fwd(const void *q, const void *k, const void *v, void *out,
                               int B, int H, int Hkv, int S, int D, int causal,
                               int block_q, int block_k, baps_stream stream)
{
    if (!out) return BAPS_ERR_INVALID_ARG;
    return baps_attention_fwd_ex(q, k, v, out, B, H, Hkv, S, D, causal, block_q, block_k,
                                 BAPS_DTYPE_BF16, nullptr, nullptr, stream);
}

baps_status baps_attention_fwd_f32(const float *q, const float *k, const float *v, float *out,
                                   int B, int H, int Hkv, int S, int D, int causal,
                                   int block_q, int block_k, baps_stream stream)
{
    if (!out) return BAPS_ERR_INVALID_ARG;
    return baps_attention_fwd_ex(q, k, v, out, B, H, Hkv, S, D, causal, block_q, block_k,
                                 BAPS_DTYPE_F32, nullptr, nullptr, stream);
}

} // extern "C"
