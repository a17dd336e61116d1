// Shared host/device plumbing of the BAPS CUDA library: status word, launch counter, checks.
#pragma once
#include <atomic>
#include <cstdint>
#include <cstdio>
#include <mutex>
#include <cuda_runtime.h>
#include "../../include/baps.h"

namespace baps {

// Device-side status word: 0 = fine; non-zero = a bounded wait expired (the value encodes
// which role gave up).  Read and cleared by baps_poll_async_error().
__device__ int g_async_status = 0;

// Host-side count of kernel launches issued by this library.
static std::atomic<int64_t> g_launches{0};

// Serialises the one-time, per-device set-up steps (table builds, symbol look-ups) when several
// host threads make their first call at the same time.
static std::mutex g_setup_mutex;

constexpr float kLog2e = 1.4426950408889634074f;

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned4(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

inline baps_status launch_status()
{
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return BAPS_ERR_CUDA;
    ++g_launches;
    return BAPS_OK;
}

inline bool have_device()
{
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev >= 0;
}

inline cudaStream_t as_stream(baps_stream s) { return reinterpret_cast<cudaStream_t>(s); }

} // namespace baps
