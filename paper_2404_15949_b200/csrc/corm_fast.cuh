// placeholder until the bf16 / head_dim 128 kernel lands
#pragma once
#include "corm_common.cuh"
namespace corm {
inline bool fast_path_available() { return false; }
inline corm_status_t launch_decode_fast(DecodeParams&, int, int, int, int, cudaStream_t) { return CORM_ERR_UNSUPPORTED; }
}
