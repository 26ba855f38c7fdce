// Tensor-core convolution path (tcgen05 / TMEM / TMA).  Placeholder interface: no layer is
// claimed yet, every convolution runs on the CUDA-core kernel.
#pragma once
#include "common.cuh"

namespace ee {

struct TcContext {};
struct TcLayer {};

inline ee_status_t tc_context_init(TcContext&) { return EE_OK; }
inline bool tc_supported(const ee_layer_desc_t&, int, int) { return false; }
inline ee_status_t tc_plan_layer(TcContext&, const ee_layer_desc_t&, int, int, int, int, int, const void*, TcLayer*) {
  return EE_ERR_UNSUPPORTED;
}
inline ee_status_t tc_launch(TcContext&, const TcLayer&, const void*, const void*, void*, int, const float*, const float*,
                             int*, cudaStream_t) {
  return EE_ERR_UNSUPPORTED;
}

}  // namespace ee
