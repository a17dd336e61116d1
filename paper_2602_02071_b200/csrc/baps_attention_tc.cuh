// placeholder until the tensor-core kernel lands
#pragma once
#include "baps_common.cuh"
namespace baps {
inline baps_status attention_tc_launch(const void *, const void *, const void *, void *, int, int, int,
                                       int, int, int, int, int, float, const baps_stats &, int,
                                       cudaStream_t)
{
    return BAPS_ERR_UNSUPPORTED;
}
} // namespace baps
