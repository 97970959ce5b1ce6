// placeholder until the tensor-core kernel lands
#pragma once
#include "common.cuh"
namespace omni {
constexpr int kTcHeads = 64;
inline omni_status_t launch_tc_decode(const DecodeParams &, cudaStream_t) { return OMNI_ERR_CUDA; }
}
