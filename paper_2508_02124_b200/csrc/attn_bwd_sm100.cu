// placeholder until the tcgen05 backward lands
#include "common.cuh"
namespace dma {
size_t tc_bwd_ws_bytes(const Prob& P) { return simt_bwd_ws_bytes(P); }
int launch_tc_bwd(const Prob& P, const void* Q, const void* K, const void* V, const void* O, const void* dO,
                  const float* lse, const float* bias, const int32_t* expiry, const uint32_t* bitmap, void* dQ,
                  void* dK, void* dV, float* dM, void* ws, cudaStream_t st) {
    return launch_simt_bwd(P, Q, K, V, O, dO, lse, bias, expiry, bitmap, dQ, dK, dV, dM, ws, st);
}
}
