// Backward of the layer (placeholder until the kernels land).
#include "l2a_common.cuh"

namespace l2a {
size_t bwd_ws_size(const l2a_params* p) { (void)p; return kWsHeaderBytes; }
}  // namespace l2a

extern "C" l2a_status l2a_backward(const l2a_params* p, const void* Q, const void* K, const void* V,
                                   const uint8_t* d_mask, const int32_t* q_idx, const int32_t* n_routed,
                                   const int32_t* prefix, const void* dO, const void* S_save, const void* A_c,
                                   const float* lse_loc, const float* lse_glb, void* dQ, void* dK, void* dV,
                                   float* dgate, void* bwd_ws, size_t bwd_ws_bytes, void* stream) {
  return L2A_ERR_UNSUPPORTED;
}
