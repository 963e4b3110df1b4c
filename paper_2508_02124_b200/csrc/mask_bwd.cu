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
    // z of every (row, head) pair of the lane group, then softplus / sigmoid ONCE per pair (the LPR lanes of a group would
    // all repeat the same forty instructions): lane `sub` takes the pairs sub, sub + LPR, ... and leaves dz and
    // dM delta softplus(z) in shared memory for the whole group
    float* sDz = sGD + G * kRows;                     // [8 warps][RPW][NR * G]
    float* sGs = sDz + 8 * RPW * NR * G;              // same shape
    float* myDz = sDz + (warp * RPW + grp) * NR * G;
    float* myGs = sGs + (warp * RPW + grp) * NR * G;
    for (int g = 0; g < G; ++g) {
        float w[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) w[c] = sW[g * D + sub * 8 + c];
#pragma unroll
        for (int n = 0; n < NR; ++n) {
            float z = 0.0f;
#pragma unroll
            for (int c = 0; c < 8; ++c) z = fmaf(v[n][c], w[c], z);
#pragma unroll
            for (int m = 1; m < LPR; m <<= 1) z += __shfl_xor_sync(0xffffffffu, z, m);
            if (sub == 0) myDz[n * G + g] = z;
        }
    }
    __syncwarp();
    for (int pr = sub; pr < NR * G; pr += LPR) {
        const int n = pr / G, g = pr % G;
        const int j = j0 + warp * RPW + n * 8 * RPW + grp;
        const float z = myDz[pr];
        const float gd = sGD[g * kRows + (j - j0)];
        const float e = __expf(-fabsf(z));                       // in (0, 1]
        const float sp = fmaxf(z, 0.0f) + log1pf(e);
        const float sig = (z >= 0.0f ? 1.0f : e) / (1.0f + e);
        myDz[pr] = gd * A[hk * G + g] * sig;
        myGs[pr] = gd * sp;
    }
    __syncwarp();
    for (int g = 0; g < G; ++g) {
        float w[8], pw[8], pa = 0.0f;
#pragma unroll
        for (int c = 0; c < 8; ++c) { w[c] = sW[g * D + sub * 8 + c]; pw[c] = 0.0f; }
#pragma unroll
        for (int n = 0; n < NR; ++n) {
            const float dz = myDz[n * G + g];
            if (sub == 0) pa += myGs[n * G + g];
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

// ---- full sampling weights: W [Hq, C], C = Hkv * D channels of the value row feed every head ----------------
// One CTA owns R consecutive keys of one batch with their whole value rows in shared memory (fp32):
//   1  z[h][row]: warp per RW rows, lanes stride the channels, W read once per warp from L2
//   2  dz[row][h] = dM delta A sigmoid(z), gs[h][row] = dM delta softplus(z)
//   3  dW partial [h][col] = sum_rows dz v: a thread owns a column and walks the rows (no cross-thread sums)
//   4  the value tile is overwritten by sum_h dz W[h][col], then added to dV
// partial [B * blocks][Hq][C + 1]; mask_bwd_full_reduce_kernel adds them in a fixed order.
constexpr int kFullThreads = 512;     // 16 warps: the kernel is bound by instruction issue and latency, not by registers

template <typename T, int RW>
__global__ void __launch_bounds__(kFullThreads) mask_bwd_full_kernel(const T* __restrict__ V, const float* __restrict__ W,
                                                                 const float* __restrict__ A, const float* __restrict__ delta,
                                                                 const float* __restrict__ dM, T* __restrict__ dV,
                                                                 float* __restrict__ partial, int L, int Hq, int Hkv, int D,
                                                                 int64_t vs_b, int64_t vs_l, int64_t vs_h) {
    constexpr int R = RW * 8;
    extern __shared__ float smem[];
    const int C = Hkv * D, HqP = (Hq + 7) & ~7;
    float* sV = smem;                              // [R][C]
    float* sDz = sV + (size_t)R * C;               // [R][HqP], heads beyond Hq hold 0
    float* sZ = sDz + (size_t)R * HqP;             // [Hq][R]: z, then dM delta softplus(z)
    const int b = blockIdx.y, j0 = blockIdx.x * R;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int C8 = C / 8, D8 = D / 8;

    for (int i = tid; i < R * C8; i += kFullThreads) {
        const int row = i / C8, ch = i % C8, j = j0 + row;
        float v[8];
        if (j < L) {
            load8f(V + b * vs_b + (int64_t)j * vs_l + (ch / D8) * vs_h + (ch % D8) * 8, v);
        } else {
#pragma unroll
            for (int c = 0; c < 8; ++c) v[c] = 0.0f;
        }
        store8f(sV + (size_t)row * C + ch * 8, v);
    }
    for (int i = tid; i < R * HqP; i += kFullThreads) sDz[i] = 0.0f;
    __syncthreads();

    // z: a warp owns HB heads at a time and all R rows; lanes stride the channels, so W is read once per CTA and each
    // value feeds HB fmas. The per-lane sums are added across lanes by a transposing butterfly (a lane keeps half of
    // its rows at each step), which leaves row (lane mod RL) of every head in the lane.
    constexpr int HB = 64 / R > 1 ? 64 / R : 1;     // 64 accumulators per thread
    constexpr int RL = R < 32 ? R : 32;            // rows reduced together
    for (int h0 = warp * HB; h0 < Hq; h0 += (kFullThreads / 32) * HB) {
        float acc[HB][R];
#pragma unroll
        for (int q = 0; q < HB; ++q)
#pragma unroll
            for (int r = 0; r < R; ++r) acc[q][r] = 0.0f;
        for (int col = lane; col < C; col += 32) {
            float w[HB];
#pragma unroll
            for (int q = 0; q < HB; ++q) w[q] = h0 + q < Hq ? __ldg(W + (size_t)(h0 + q) * C + col) : 0.0f;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float v = sV[(size_t)r * C + col];
#pragma unroll
                for (int q = 0; q < HB; ++q) acc[q][r] = fmaf(v, w[q], acc[q][r]);
            }
        }
#pragma unroll
        for (int q = 0; q < HB; ++q) {
#pragma unroll
            for (int base = 0; base < R; base += RL) {
#pragma unroll
                for (int keep = RL >> 1; keep >= 1; keep >>= 1) {
                    const bool up = (lane & keep) != 0;
#pragma unroll
                    for (int r = 0; r < keep; ++r) {
                        const float stay = up ? acc[q][base + r + keep] : acc[q][base + r];
                        const float give = up ? acc[q][base + r] : acc[q][base + r + keep];
                        acc[q][base + r] = stay + __shfl_xor_sync(0xffffffffu, give, keep);
                    }
                }
#pragma unroll
                for (int m = RL; m < 32; m <<= 1) acc[q][base] += __shfl_xor_sync(0xffffffffu, acc[q][base], m);
                if (lane < RL && h0 + q < Hq) sZ[(h0 + q) * R + base + lane] = acc[q][base];
            }
        }
    }
    __syncthreads();

    for (int i = tid; i < Hq * R; i += kFullThreads) {
        const int h = i / R, row = i % R, j = j0 + row;
        float dz = 0.0f, gs = 0.0f;
        if (j < L) {
            const size_t at = ((size_t)b * Hq + h) * L + j;
            const float gd = dM[at] * delta[at];
            const float z = sZ[i];
            const float e = __expf(-fabsf(z));
            gs = gd * (fmaxf(z, 0.0f) + log1pf(e));
            dz = gd * A[h] * ((z >= 0.0f ? 1.0f : e) / (1.0f + e));
        }
        sDz[row * HqP + h] = dz;
        sZ[i] = gs;
    }
    __syncthreads();

    float* out = partial + ((size_t)b * gridDim.x + blockIdx.x) * Hq * (C + 1);
    for (int col = tid; col < C; col += kFullThreads) {
        for (int hc = 0; hc < HqP; hc += 8) {
            float acc[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) acc[q] = 0.0f;
            for (int row = 0; row < R; ++row) {
                const float v = sV[(size_t)row * C + col];
                const float4 a = *reinterpret_cast<const float4*>(sDz + row * HqP + hc);
                const float4 c = *reinterpret_cast<const float4*>(sDz + row * HqP + hc + 4);
                acc[0] = fmaf(a.x, v, acc[0]); acc[1] = fmaf(a.y, v, acc[1]); acc[2] = fmaf(a.z, v, acc[2]); acc[3] = fmaf(a.w, v, acc[3]);
                acc[4] = fmaf(c.x, v, acc[4]); acc[5] = fmaf(c.y, v, acc[5]); acc[6] = fmaf(c.z, v, acc[6]); acc[7] = fmaf(c.w, v, acc[7]);
            }
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (hc + q < Hq) out[(size_t)(hc + q) * (C + 1) + col] = acc[q];
        }
    }
    if (tid < Hq) {
        float t = 0.0f;
        for (int row = 0; row < R; ++row) t += sZ[tid * R + row];
        out[(size_t)tid * (C + 1) + C] = t;
    }
    __syncthreads();   // every thread is done with the values of its columns' neighbours: the tile may be overwritten

    for (int col = tid; col < C; col += kFullThreads) {
        for (int hc = 0; hc < HqP; hc += 8) {
            float w[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) w[q] = hc + q < Hq ? __ldg(W + (size_t)(hc + q) * C + col) : 0.0f;
            for (int row = 0; row < R; ++row) {
                const float4 a = *reinterpret_cast<const float4*>(sDz + row * HqP + hc);
                const float4 c = *reinterpret_cast<const float4*>(sDz + row * HqP + hc + 4);
                float u = a.x * w[0];
                u = fmaf(a.y, w[1], u); u = fmaf(a.z, w[2], u); u = fmaf(a.w, w[3], u);
                u = fmaf(c.x, w[4], u); u = fmaf(c.y, w[5], u); u = fmaf(c.z, w[6], u); u = fmaf(c.w, w[7], u);
                float* dst = sV + (size_t)row * C + col;
                *dst = hc == 0 ? u : *dst + u;
            }
        }
    }
    __syncthreads();

    for (int i = tid; i < R * C8; i += kFullThreads) {
        const int row = i / C8, ch = i % C8, j = j0 + row;
        if (j < L) {
            T* p = dV + b * vs_b + (int64_t)j * vs_l + (ch / D8) * vs_h + (ch % D8) * 8;
            float cur[8];
            load8f(p, cur);
#pragma unroll
            for (int c = 0; c < 8; ++c) cur[c] += sV[(size_t)row * C + ch * 8 + c];
            store8f(p, cur);
        }
    }
}

// dW [Hq][C] and dA [Hq] from partial [n][Hq][C + 1]: four groups of threads each add every fourth partial in index order,
// then the group sums are added in group order.
__global__ void __launch_bounds__(512) mask_bwd_full_reduce_kernel(const float* __restrict__ partial, float* __restrict__ dW,
                                                                   float* __restrict__ dA, int n, int Hq, int C) {
    __shared__ float part[4][128];
    const int h = blockIdx.y, c = blockIdx.x * 128 + (threadIdx.x & 127), grp = threadIdx.x >> 7;
    float s = 0.0f;
    if (c <= C)
        for (int t = grp; t < n; t += 4) s += partial[((size_t)t * Hq + h) * (C + 1) + c];
    part[grp][threadIdx.x & 127] = s;
    __syncthreads();
    if (grp == 0 && c <= C) {
        const float tot = ((part[0][threadIdx.x] + part[1][threadIdx.x]) + part[2][threadIdx.x]) + part[3][threadIdx.x];
        if (c < C) dW[(size_t)h * C + c] = tot; else dA[h] = tot;
    }
}

// rows per CTA: the largest of 64, 32, 16, 8 whose tile fits 200 KiB of shared memory (0: none does)
static int full_rows(const Prob& P) {
    const size_t C = (size_t)P.Hkv * P.d, HqP = (P.Hq + 7) & ~7;
    for (int R = 64; R >= 8; R >>= 1)
        if ((R * C + R * HqP + (size_t)P.Hq * R) * sizeof(float) <= 200 * 1024) return R;
    return 0;
}

}  // namespace

size_t mask_bwd_ws_bytes(const Prob& P) {
    if (P.flags & DMA_FLAG_FULL_DELTA) {
        const int R = full_rows(P);
        if (R == 0) return 0;
        return (size_t)P.B * ((P.L + R - 1) / R) * P.Hq * ((size_t)P.Hkv * P.d + 1) * sizeof(float);
    }
    const size_t nblk = (size_t)(P.L + kRows - 1) / kRows;
    return (size_t)P.B * P.Hkv * nblk * P.G * (P.d + 1) * sizeof(float);
}

template <typename T, int D>
static int launch_typed(const Prob& P, const void* V, const float* W, const float* A, const float* delta, const float* dM,
                        void* dV, float* dW, float* dA, void* ws, cudaStream_t st) {
    const int nblk = (P.L + kRows - 1) / kRows;
    const size_t smem = (size_t)P.G * (D + 8 * (D + 1) + 3 * kRows) * sizeof(float);
    if (cudaFuncSetAttribute(mask_bwd_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DMA_ERR_CUDA;
    mask_bwd_kernel<T, D><<<dim3(nblk, P.Hkv, P.B), kThreads, smem, st>>>((const T*)V, W, A, delta, dM, (T*)dV, (float*)ws, P.L, P.Hq,
                                                                            P.G, P.vs[0], P.vs[1], P.vs[2]);
    mask_bwd_reduce_kernel<D><<<P.Hq, (D == 128 ? 4 : 8) * (D + 1), 0, st>>>((const float*)ws, dW, dA, P.B, P.Hkv, P.G, nblk);
    count_launch(2);
    return check_launch();
}

template <typename T, int RW>
static int launch_full(const Prob& P, const void* V, const float* W, const float* A, const float* delta, const float* dM,
                       void* dV, float* dW, float* dA, void* ws, cudaStream_t st) {
    constexpr int R = RW * 8;
    const int nblk = (P.L + R - 1) / R, C = P.Hkv * P.d, HqP = (P.Hq + 7) & ~7;
    const size_t smem = ((size_t)R * C + (size_t)R * HqP + (size_t)P.Hq * R) * sizeof(float);
    if (cudaFuncSetAttribute(mask_bwd_full_kernel<T, RW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return DMA_ERR_CUDA;
    mask_bwd_full_kernel<T, RW><<<dim3(nblk, P.B), kFullThreads, smem, st>>>((const T*)V, W, A, delta, dM, (T*)dV, (float*)ws, P.L, P.Hq,
                                                                          P.Hkv, P.d, P.vs[0], P.vs[1], P.vs[2]);
    mask_bwd_full_reduce_kernel<<<dim3((C + 1 + 127) / 128, P.Hq), 512, 0, st>>>((const float*)ws, dW, dA, P.B * nblk, P.Hq, C);
    count_launch(2);
    return check_launch();
}

template <typename T>
static int launch_full_rows(const Prob& P, const void* V, const float* W, const float* A, const float* delta, const float* dM,
                            void* dV, float* dW, float* dA, void* ws, cudaStream_t st) {
    switch (full_rows(P)) {
        case 64: return launch_full<T, 8>(P, V, W, A, delta, dM, dV, dW, dA, ws, st);
        case 32: return launch_full<T, 4>(P, V, W, A, delta, dM, dV, dW, dA, ws, st);
        case 16: return launch_full<T, 2>(P, V, W, A, delta, dM, dV, dW, dA, ws, st);
        case 8: return launch_full<T, 1>(P, V, W, A, delta, dM, dV, dW, dA, ws, st);
    }
    return DMA_ERR_UNSUPPORTED;
}

int launch_mask_bwd(const Prob& P, const void* V, const float* W, const float* A, const float* delta, const float* dM,
                    void* dV, float* dW, float* dA, void* ws, cudaStream_t st) {
    if (P.flags & DMA_FLAG_FULL_DELTA)
        return P.dtype == DMA_BF16 ? launch_full_rows<__nv_bfloat16>(P, V, W, A, delta, dM, dV, dW, dA, ws, st)
                                   : launch_full_rows<float>(P, V, W, A, delta, dM, dV, dW, dA, ws, st);
    if (P.G > 16) return DMA_ERR_UNSUPPORTED;
    if (P.dtype == DMA_BF16) {
        return P.d == 128 ? launch_typed<__nv_bfloat16, 128>(P, V, W, A, delta, dM, dV, dW, dA, ws, st)
                          : launch_typed<__nv_bfloat16, 64>(P, V, W, A, delta, dM, dV, dW, dA, ws, st);
    }
    return P.d == 128 ? launch_typed<float, 128>(P, V, W, A, delta, dM, dV, dW, dA, ws, st)
                      : launch_typed<float, 64>(P, V, W, A, delta, dM, dV, dW, dA, ws, st);
}

}  // namespace dma
