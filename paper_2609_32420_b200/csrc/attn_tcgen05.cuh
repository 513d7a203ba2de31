// placeholder until the tcgen05 kernel lands
#pragma once
#include "common.cuh"
#include "attn_portable.cuh"
namespace carnator {
inline bool tcgen05_supported(const carnator_shape*) { return false; }
inline carnator_status launch_tcgen05(const AttnArgs&, const carnator_shape*, cudaStream_t, char*, size_t, long long*) {
    return CARNATOR_ERR_UNSUPPORTED;
}
}
