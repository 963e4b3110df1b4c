// bf16 tensors with 64 channels run on the 128-channel tensor-core kernels through zero-padded copies: with the upper 64
// channels of Q, K, V (and O, dO) zero, S = Q K^T, P, dP and D are unchanged and the upper channels of O, dQ, dK, dV come
// out zero, so the kernels compute exactly the 64-channel problem (at twice its tensor work, still far from the CUDA-core
// kernels' time). These two kernels copy between a strided [B, L, H, 64] tensor and a packed [B, L, H, 128] one.
#include "common.cuh"

namespace dma {
namespace {

// one thread per 16-byte chunk of a padded row (16 chunks per row: 8 copied, 8 zero)
__global__ void __launch_bounds__(256) pad64_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst,
                                                    size_t rows, int L, int H, int64_t s_b, int64_t s_l, int64_t s_h) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t row = idx >> 4;
    const int c = (int)(idx & 15);
    if (row >= rows) return;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (c < 8) {
        const int h = (int)(row % H), l = (int)((row / H) % L);
        const int64_t b = (int64_t)(row / ((size_t)H * L));
        v = *reinterpret_cast<const uint4*>(src + b * s_b + (int64_t)l * s_l + (int64_t)h * s_h + c * 8);
    }
    *reinterpret_cast<uint4*>(dst + row * 128 + c * 8) = v;
}

// one thread per 16-byte chunk of the 64 kept channels
__global__ void __launch_bounds__(256) unpad64_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst,
                                                      size_t rows, int L, int H, int64_t s_b, int64_t s_l, int64_t s_h) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t row = idx >> 3;
    const int c = (int)(idx & 7);
    if (row >= rows) return;
    const int h = (int)(row % H), l = (int)((row / H) % L);
    const int64_t b = (int64_t)(row / ((size_t)H * L));
    *reinterpret_cast<uint4*>(dst + b * s_b + (int64_t)l * s_l + (int64_t)h * s_h + c * 8) =
        *reinterpret_cast<const uint4*>(src + row * 128 + c * 8);
}

}  // namespace

int launch_pad64(const void* src, void* dst, int B, int L, int H, const int64_t (&s)[3], cudaStream_t st) {
    const size_t rows = (size_t)B * L * H;
    pad64_kernel<<<(unsigned)((rows * 16 + 255) / 256), 256, 0, st>>>((const __nv_bfloat16*)src, (__nv_bfloat16*)dst, rows, L, H, s[0],
                                                                      s[1], s[2]);
    count_launch();
    return check_launch();
}

int launch_unpad64(const void* src, void* dst, int B, int L, int H, const int64_t (&s)[3], cudaStream_t st) {
    const size_t rows = (size_t)B * L * H;
    unpad64_kernel<<<(unsigned)((rows * 8 + 255) / 256), 256, 0, st>>>((const __nv_bfloat16*)src, (__nv_bfloat16*)dst, rows, L, H, s[0],
                                                                       s[1], s[2]);
    count_launch();
    return check_launch();
}

}  // namespace dma
