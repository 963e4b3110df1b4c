// Mask-generation backward (Sec. 4.3: the bias gradient dM flows on to the sampling weights W_delta and the gate A;
// Eq. delta_calc differentiated, the top-w selection held fixed):
//   z = v . W_h, sp = softplus(z), delta = exp(A_h sp)   (delta is taken from the forward's bias output)
//   g = dM delta;  dA_h = sum g sp;  dz = g A_h sigmoid(z);  dW_h = sum dz v;  dV[j, kv head] += sum_h dz W_h
// HBM-bound: V and dV rows are read once, dV written once. One CTA owns 64 consecutive keys of one (batch, KV head)
// and all G query heads of the group; dW / dA partial sums go to the workspace and a second kernel adds them in a
// fixed order (no floating-point atomics: the result does not depend on the launch schedule).
#include "common.cuh"

namespace dma {
namespace {

constexpr int kRows = 64;      // keys per CTA
constexpr int kThreads = 256;

__device__ __forceinline__ void load8f(const float* p, float (&v)[8]) {
    const float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8f(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 a = *reinterpret_cast<const uint4*>(p);
    const uint32_t u[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(u[i] << 16);
        v[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ void store8f(float* p, const float (&v)[8]) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(p + 4) = make_float4(v[4], v[5], v[6], v[7]);
}
__device__ __forceinline__ void store8f(__nv_bfloat16* p, const float (&v)[8]) {
    uint4 o;
    o.x = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v[0])) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v[1])) << 16);
    o.y = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v[2])) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v[3])) << 16);
    o.z = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v[4])) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v[5])) << 16);
    o.w = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v[6])) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v[7])) << 16);
    *reinterpret_cast<uint4*>(p) = o;
}

// A group of D/8 lanes owns a key row (8 channels per lane); each thread keeps its rows of V and of the dV update in
// registers while the query heads of the group are walked, so V is read exactly once.
// partial [blocks][G][D + 1]: per CTA the sums over its keys of dz v (D values) and of g sp (1 value).
template <typename T, int D>
__global__ void __launch_bounds__(kThreads) mask_bwd_kernel(const T* __restrict__ V, const float* __restrict__ W,
                                                            const float* __restrict__ A, const float* __restrict__ delta,
                                                            const float* __restrict__ dM, T* __restrict__ dV,
                                                            float* __restrict__ partial, int L, int Hq, int G,
                                                            int64_t vs_b, int64_t vs_l, int64_t vs_h) {
    constexpr int LPR = D / 8;                       // lanes per row
    constexpr int RPW = 32 / LPR;                    // rows per warp and pass
    constexpr int NR = kRows / (8 * RPW);            // rows per thread
    extern __shared__ float smem[];
    float* sW = smem;                                // [G][D]
    float* sAcc = smem + G * D;                      // [8 warps][G][D + 1]
    const int hk = blockIdx.y, b = blockIdx.z, j0 = blockIdx.x * kRows;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LPR, grp = lane / LPR;
    float* sGD = sAcc + 8 * G * (D + 1);             // [G][kRows]: dM * delta of the CTA's keys, fetched in one batch
    for (int i = tid; i < G * D; i += kThreads) sW[i] = W[(size_t)hk * G * D + i];
    for (int i = tid; i < G * kRows; i += kThreads) {
        const int g = i / kRows, j = j0 + i % kRows;
        const size_t at = ((size_t)b * Hq + hk * G + g) * L + j;
        sGD[i] = j < L ? dM[at] * delta[at] : 0.0f;
    }
    __syncthreads();

    float v[NR][8], upd[NR][8];
#pragma unroll
    for (int n = 0; n < NR; ++n) {
        const int j = j0 + warp * RPW + n * 8 * RPW + grp;
        if (j < L) {
            load8f(V + b * vs_b + (int64_t)j * vs_l + hk * vs_h + sub * 8, v[n]);
        } else {
#pragma unroll
            for (int c = 0; c < 8; ++c) v[n][c] = 0.0f;
        }
#pragma unroll
        for (int c = 0; c < 8; ++c) upd[n][c] = 0.0f;
    }
    for (int g = 0; g < G; ++g) {
        const int h = hk * G + g;
        const float a = A[h];
        float w[8], pw[8], pa = 0.0f;
#pragma unroll
        for (int c = 0; c < 8; ++c) { w[c] = sW[g * D + sub * 8 + c]; pw[c] = 0.0f; }
#pragma unroll
        for (int n = 0; n < NR; ++n) {
            const int j = j0 + warp * RPW + n * 8 * RPW + grp;
            float z = 0.0f;
#pragma unroll
            for (int c = 0; c < 8; ++c) z = fmaf(v[n][c], w[c], z);
#pragma unroll
            for (int m = 1; m < LPR; m <<= 1) z += __shfl_xor_sync(0xffffffffu, z, m);
            const float gd = sGD[g * kRows + (j - j0)];
            const float e = __expf(-fabsf(z));                       // in (0, 1]
            const float sp = fmaxf(z, 0.0f) + log1pf(e);
            const float sig = (z >= 0.0f ? 1.0f : e) / (1.0f + e);
            const float dz = gd * a * sig;
            if (sub == 0) pa += gd * sp;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                pw[c] = fmaf(dz, v[n][c], pw[c]);
                upd[n][c] = fmaf(dz, w[c], upd[n][c]);
            }
        }
        // lanes with the same channel slice (the RPW row groups of the warp) are added by shuffles, then each warp
        // leaves its sums in its own shared-memory slice; the slices are added in warp order below
#pragma unroll
        for (int m = LPR; m < 32; m <<= 1) {
#pragma unroll
            for (int c = 0; c < 8; ++c) pw[c] += __shfl_xor_sync(0xffffffffu, pw[c], m);
            pa += __shfl_xor_sync(0xffffffffu, pa, m);
        }
        if (grp == 0) {
            float* dst = sAcc + ((size_t)warp * G + g) * (D + 1);
#pragma unroll
            for (int c = 0; c < 8; ++c) dst[sub * 8 + c] = pw[c];
            if (sub == 0) dst[D] = pa;
        }
    }
#pragma unroll
    for (int n = 0; n < NR; ++n) {
        const int j = j0 + warp * RPW + n * 8 * RPW + grp;
        if (j < L) {
            T* p = dV + b * vs_b + (int64_t)j * vs_l + hk * vs_h + sub * 8;
            float cur[8];
            load8f(p, cur);
#pragma unroll
            for (int c = 0; c < 8; ++c) cur[c] += upd[n][c];
            store8f(p, cur);
        }
    }
    __syncthreads();
    const size_t blk = ((size_t)b * gridDim.y + hk) * gridDim.x + blockIdx.x;
    for (int i = tid; i < G * (D + 1); i += kThreads) {
        float t = 0.0f;
#pragma unroll
        for (int wq = 0; wq < 8; ++wq) t += sAcc[(size_t)wq * G * (D + 1) + i];
        partial[blk * G * (D + 1) + i] = t;
    }
}

// dW[h][c] and dA[h]: sum of the per-CTA partials over batches and key blocks. kGroups groups of threads each add every
// kGroups-th partial in index order, then the group sums are added in group order: a fixed order, whatever the schedule.
template <int D>
__global__ void __launch_bounds__((D == 128 ? 4 : 8) * (D + 1)) mask_bwd_reduce_kernel(const float* __restrict__ partial, float* __restrict__ dW,
                                                                     float* __restrict__ dA, int B, int Hkv, int G, int nblk) {
    constexpr int kGroups = D == 128 ? 4 : 8;      // kGroups * (D + 1) threads <= 1024
    __shared__ float part[kGroups][D + 1];
    const int h = blockIdx.x, hk = h / G, g = h % G;
    const int c = threadIdx.x % (D + 1), grp = threadIdx.x / (D + 1);
    float s = 0.0f;
    const int total = B * nblk;
    for (int t = grp; t < total; t += kGroups) {
        const int b = t / nblk, k = t % nblk;
        s += partial[((((size_t)b * Hkv + hk) * nblk + k) * G + g) * (D + 1) + c];
    }
    part[grp][c] = s;
    __syncthreads();
    if (grp == 0) {
        float tot = 0.0f;
#pragma unroll
        for (int q = 0; q < kGroups; ++q) tot += part[q][c];
        if (c < D) dW[(size_t)h * D + c] = tot; else dA[h] = tot;
    }
}

}  // namespace

size_t mask_bwd_ws_bytes(const Prob& P) {
    const size_t nblk = (size_t)(P.L + kRows - 1) / kRows;
    return (size_t)P.B * P.Hkv * nblk * P.G * (P.d + 1) * sizeof(float);
}

template <typename T, int D>
static int launch_typed(const Prob& P, const void* V, const float* W, const float* A, const float* delta, const float* dM,
                        void* dV, float* dW, float* dA, void* ws, cudaStream_t st) {
    const int nblk = (P.L + kRows - 1) / kRows;
    const size_t smem = (size_t)P.G * (D + 8 * (D + 1) + kRows) * sizeof(float);
    if (cudaFuncSetAttribute(mask_bwd_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DMA_ERR_CUDA;
    mask_bwd_kernel<T, D><<<dim3(nblk, P.Hkv, P.B), kThreads, smem, st>>>((const T*)V, W, A, delta, dM, (T*)dV, (float*)ws, P.L, P.Hq,
                                                                            P.G, P.vs[0], P.vs[1], P.vs[2]);
    mask_bwd_reduce_kernel<D><<<P.Hq, (D == 128 ? 4 : 8) * (D + 1), 0, st>>>((const float*)ws, dW, dA, P.B, P.Hkv, P.G, nblk);
    count_launch(2);
    return check_launch();
}

int launch_mask_bwd(const Prob& P, const void* V, const float* W, const float* A, const float* delta, const float* dM,
                    void* dV, float* dW, float* dA, void* ws, cudaStream_t st) {
    if (P.G > 16) return DMA_ERR_UNSUPPORTED;
    if (P.dtype == DMA_BF16) {
        return P.d == 128 ? launch_typed<__nv_bfloat16, 128>(P, V, W, A, delta, dM, dV, dW, dA, ws, st)
                          : launch_typed<__nv_bfloat16, 64>(P, V, W, A, delta, dM, dV, dW, dA, ws, st);
    }
    return P.d == 128 ? launch_typed<float, 128>(P, V, W, A, delta, dM, dV, dW, dA, ws, st)
                      : launch_typed<float, 64>(P, V, W, A, delta, dM, dV, dW, dA, ws, st);
}

}  // namespace dma
