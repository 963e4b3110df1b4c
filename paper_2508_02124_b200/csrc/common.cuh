// Shared declarations of the DMA CUDA library: resolved problem view, launch accounting, small device helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dma.h"

namespace dma {

constexpr int kWsHeaderBytes = 256;   // every workspace starts with this header; int32 word 0 = status

// dma_problem_t with defaults resolved and derived sizes filled in.
struct Prob {
    int B, Hq, Hkv, L, d, G;
    int w;                 // min(w, L)
    int w_cap;             // w as given (the capacity of an incremental decoding state)
    int dtype, flags;
    int causal;            // 1: key j visible to rows i >= j; 0: to every row (the key's first row is 0 instead of j)
    int bm, bn, Tr, Tc, Wd;   // bitmap tile sizes, tile counts, uint32 words per bitmap row
    int Lq, q_off;            // forward over a chunk of query rows: Q, O, lse hold the rows q_off .. q_off + Lq - 1 (Lq = L, q_off = 0: all)
    float scale;
    int64_t qs[3], ks[3], vs[3], os[3];   // batch, seq, head strides in elements
};

int resolve(const dma_problem_t* p, Prob* out);          // validation + defaults; returns dma_status
void count_launch(int n = 1);
// measurement hook (dma_kernel_timing): brackets a stage's main kernel with a pair of CUDA events while recording is on
void timing_mark(int which, bool after, cudaStream_t st);
int check_launch();                                       // cudaGetLastError -> dma_status

// stage launchers (each returns a dma_status); defined in the stage's .cu file
size_t mask_ws_bytes(const Prob& P);
size_t mask_bwd_ws_bytes(const Prob& P);
int launch_delta_range(const Prob& P, const void* V, const float* W, const float* A, float* delta, int64_t ld, int j_begin,
                       int j_end, cudaStream_t st);
size_t decode_ws_bytes(const Prob& P);
size_t decode_state_bytes(const Prob& P);
int launch_decode_state_init(const Prob& P, const float* delta, int64_t ld, int* state, void* ws, cudaStream_t st);
int launch_decode_step(const Prob& P, const void* q, const void* K, const void* V, const float* delta, int64_t ld, int* state,
                       void* o, float* lse, void* ws, cudaStream_t st);
int launch_decode(const Prob& P, const void* q, const void* K, const void* V, const float* delta, int64_t ld, void* o, float* lse,
                  int32_t* sel_idx, void* ws, cudaStream_t st);
int launch_mask_bwd(const Prob& P, const void* V, const float* W, const float* A, const float* delta, const float* dM,
                    void* dV, float* dW, float* dA, void* ws, cudaStream_t st);
int launch_mask_build(const Prob& P, const void* V, const float* W, const float* A, float* bias, int32_t* expiry,
                      uint32_t* bitmap, void* ws, cudaStream_t st, const int32_t* cu_seqlens = nullptr, int nseq = 0);

size_t simt_bwd_ws_bytes(const Prob& P);
int launch_simt_fwd(const Prob& P, const void* Q, const void* K, const void* V, const float* bias,
                    const int32_t* expiry, const uint32_t* bitmap, void* O, float* lse, cudaStream_t st);
int launch_simt_bwd(const Prob& P, const void* Q, const void* K, const void* V, const void* O, const void* dO,
                    const float* lse, const float* bias, const int32_t* expiry, const uint32_t* bitmap, void* dQ,
                    void* dK, void* dV, float* dM, void* ws, cudaStream_t st);

size_t tc_fwd_ws_bytes(const Prob& P);
int launch_tc_fwd(const Prob& P, const void* Q, const void* K, const void* V, const float* bias,
                  const int32_t* expiry, const uint32_t* bitmap, void* O, float* lse, void* ws, cudaStream_t st);
size_t tc_bwd_ws_bytes(const Prob& P);
int launch_tc_bwd(const Prob& P, const void* Q, const void* K, const void* V, const void* O, const void* dO,
                  const float* lse, const float* bias, const int32_t* expiry, const uint32_t* bitmap, void* dQ,
                  void* dK, void* dV, float* dM, void* ws, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void store_as(float* p, float x) { *p = x; }
__device__ __forceinline__ void store_as(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

// bit (kt % 32) of word [bh, qt, kt / 32]
__device__ __forceinline__ bool bitmap_test(const uint32_t* bitmap, int Tr, int Wd, int bh, int qt, int kt) {
    return (bitmap[((size_t)bh * Tr + qt) * Wd + (kt >> 5)] >> (kt & 31)) & 1u;
}

}  // namespace dma
