// The table of w0(u) = HiF8(2^HiF8(u)) in global memory, built once per device (its entries take
// the exponential in double precision, too slow to repeat in every CTA); the kernels copy it into
// shared memory.
#pragma once
#include "baps_common.cuh"
#include "baps_hif8.cuh"

namespace baps {

__device__ float g_w0_table[kLutN];

__global__ void w0_table_init_kernel()
{
    for (int i = threadIdx.x; i < kLutN; i += blockDim.x) g_w0_table[i] = w0_table_entry(i);
}

// First call on a device: fill the table and wait for it (later calls may come on any stream).
// (Internal linkage: the "table is ready" record must belong to this copy of the library alone -- a
// function-local static of a plain inline function would be shared with any other copy loaded into
// the process, whose own device table would then never be built.)
static inline baps_status ensure_w0_table(cudaStream_t stream)
{
    static bool table_ready[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BAPS_ERR_CUDA;
    std::lock_guard<std::mutex> setup_lock(g_setup_mutex);
    if (!table_ready[dev]) {
        w0_table_init_kernel<<<1, 320, 0, stream>>>();
        if (cudaGetLastError() != cudaSuccess) return BAPS_ERR_CUDA;
        ++g_launches;
        if (cudaStreamSynchronize(stream) != cudaSuccess) return BAPS_ERR_CUDA;
        table_ready[dev] = true;
    }
    return BAPS_OK;
}

} // namespace baps
