// CUDA-core (fp32 FMA) attention kernels: the fp32 element type needs full fp32 products, which the tensor
// cores do not give. Same semantics as the tensor-core path: additive per-key bias, per-element validity
// j <= i < expiry[j], key tiles whose bitmap bit is clear are neither loaded nor computed.
//   forward   Alg. 1 with the loop order swapped (one CTA owns a query tile, online softmax across key tiles)
//   backward  Alg. 2: one CTA owns a key tile of one KV head, walks the query heads of the group and their
//             active query tiles, keeps dK/dV in registers, reduces dM per column, adds dQ with atomics
#include "common.cuh"

namespace dma {
namespace {

constexpr int BM = 64, BN = 64, NT = 256;

template <typename T>
__device__ __forceinline__ void load_tile(float* dst, int ld, const T* src, int64_t row_stride, int r0, int L, int D) {
    // rows r0..r0+63 (zero beyond L), D contiguous channels each
    for (int idx = threadIdx.x; idx < 64 * D; idx += NT) {
        int r = idx / D, c = idx % D;
        dst[r * ld + c] = (r0 + r < L) ? to_f32(src[(int64_t)(r0 + r) * row_stride + c]) : 0.0f;
    }
}

template <typename T, int D>
__global__ void __launch_bounds__(NT) simt_fwd_kernel(const T* __restrict__ Q, const T* __restrict__ K,
                                                      const T* __restrict__ V, const float* __restrict__ bias,
                                                      const int32_t* __restrict__ expiry,
                                                      const uint32_t* __restrict__ bitmap, T* __restrict__ O,
                                                      float* __restrict__ lse, Prob P, int use_bitmap) {
    constexpr int LDQ = D + 1, LDS = BN + 1;
    extern __shared__ float sm[];
    float* sQ = sm;                    // [BM][LDQ]
    float* sK = sQ + BM * LDQ;         // [BN][LDQ]
    float* sV = sK + BN * LDQ;         // [BN][D]
    float* sS = sV + BN * D;           // [BM][LDS]
    float* sM = sS + BM * LDS;         // running max      [BM]
    float* sL = sM + BM;               // running sum      [BM]
    float* sA = sL + BM;               // rescale factor   [BM]
    float* sB = sA + BM;               // bias of the tile [BN]
    int* sE = reinterpret_cast<int*>(sB + BN);   // expiry of the tile [BN]

    const int qt = blockIdx.x, h = blockIdx.y, b = blockIdx.z, hk = h / P.G, bh = b * P.Hq + h;
    const int i0 = qt * BM, L = P.L;                 // i0: first row of the tile inside the chunk; row i0 + r is position ia0 + r
    const int ia0 = P.q_off + i0;
    const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
    const T* q = Q + b * P.qs[0] + h * P.qs[2];
    const T* k = K + b * P.ks[0] + hk * P.ks[2];
    const T* v = V + b * P.vs[0] + hk * P.vs[2];

    load_tile(sQ, LDQ, q, P.qs[1], i0, P.Lq, D);
    if (tid < BM) { sM[tid] = -INFINITY; sL[tid] = 0.0f; }
    float acc[4][D / 16];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < D / 16; ++c) acc[a][c] = 0.0f;

    const int last = P.causal ? min(ia0 + BM, L) - 1 : L - 1;  // last key any row of the tile can see
    for (int j0 = 0; j0 <= last; j0 += BN) {
        if (use_bitmap && !bitmap_test(bitmap, P.Tr, P.Wd, bh, ia0 / P.bm, j0 / P.bn)) continue;
        __syncthreads();
        load_tile(sK, LDQ, k, P.ks[1], j0, L, D);
        load_tile(sV, D, v, P.vs[1], j0, L, D);
        if (tid < BN) {
            int j = j0 + tid;
            sB[tid] = j < L ? bias[(size_t)bh * L + j] : 0.0f;
            sE[tid] = j < L ? expiry[(size_t)bh * L + j] : 0;
        }
        __syncthreads();
        float s[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int c = 0; c < 4; ++c) s[a][c] = 0.0f;
        for (int kk = 0; kk < D; ++kk) {
            float qa[4], kb[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) qa[a] = sQ[(ty + 16 * a) * LDQ + kk];
#pragma unroll
            for (int c = 0; c < 4; ++c) kb[c] = sK[(tx + 16 * c) * LDQ + kk];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int c = 0; c < 4; ++c) s[a][c] = fmaf(qa[a], kb[c], s[a][c]);
        }
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                int r = ty + 16 * a, cc = tx + 16 * c, i = ia0 + r, j = j0 + cc;
                bool ok = (j <= i || !P.causal) && i < sE[cc];
                sS[r * LDS + cc] = ok ? s[a][c] * P.scale + sB[cc] : -INFINITY;
            }
        __syncthreads();
        {   // online softmax: 4 threads per row, 16 columns each
            int r = tid / 4, part = tid % 4;
            float mx = -INFINITY;
            for (int c = part * 16; c < part * 16 + 16; ++c) mx = fmaxf(mx, sS[r * LDS + c]);
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            float m_old = sM[r], m_new = fmaxf(m_old, mx);
            float m_use = m_new == -INFINITY ? 0.0f : m_new;
            float sum = 0.0f;
            for (int c = part * 16; c < part * 16 + 16; ++c) {
                float p = __expf(sS[r * LDS + c] - m_use);
                sS[r * LDS + c] = p;
                sum += p;
            }
            sum += __shfl_xor_sync(0xffffffffu, sum, 1);
            sum += __shfl_xor_sync(0xffffffffu, sum, 2);
            if (part == 0) {
                float alpha = __expf(m_old - m_use);
                sA[r] = alpha;
                sL[r] = sL[r] * alpha + sum;
                sM[r] = m_new;
            }
        }
        __syncthreads();
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            float alpha = sA[ty + 16 * a];
#pragma unroll
            for (int c = 0; c < D / 16; ++c) acc[a][c] *= alpha;
        }
        for (int j = 0; j < BN; ++j) {
            float pa[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) pa[a] = sS[(ty + 16 * a) * LDS + j];
#pragma unroll
            for (int c = 0; c < D / 16; ++c) {
                float vv = sV[j * D + tx + 16 * c];
#pragma unroll
                for (int a = 0; a < 4; ++a) acc[a][c] = fmaf(pa[a], vv, acc[a][c]);
            }
        }
    }
    __syncthreads();
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        int r = ty + 16 * a, i = i0 + r;
        if (i >= P.Lq) continue;
        float l = sL[r], inv = l > 0.0f ? 1.0f / l : 0.0f;
        T* o = O + b * P.os[0] + (int64_t)i * P.os[1] + h * P.os[2];
#pragma unroll
        for (int c = 0; c < D / 16; ++c) store_as(o + tx + 16 * c, acc[a][c] * inv);
        if (tx == 0) lse[(size_t)bh * P.Lq + i] = l > 0.0f ? sM[r] + logf(l) : -INFINITY;
    }
}

// D_i = dO_i . O_i  (Alg. 2): one warp per (b, h, i)
template <typename T>
__global__ void rowdot_kernel(const T* __restrict__ O, const T* __restrict__ dO, float* __restrict__ Dv, Prob P) {
    const long row = (long)blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
    const int lane = threadIdx.x % 32;
    if (row >= (long)P.B * P.Hq * P.L) return;
    const int i = row % P.L, h = (row / P.L) % P.Hq, b = row / ((long)P.L * P.Hq);
    const T* o = O + b * P.os[0] + (int64_t)i * P.os[1] + h * P.os[2];
    const T* g = dO + b * P.os[0] + (int64_t)i * P.os[1] + h * P.os[2];
    float s = 0.0f;
    for (int c = lane; c < P.d; c += 32) s = fmaf(to_f32(o[c]), to_f32(g[c]), s);
    for (int m = 16; m; m >>= 1) s += __shfl_xor_sync(0xffffffffu, s, m);
    if (lane == 0) Dv[row] = s;
}

template <typename T, int D>
__global__ void __launch_bounds__(NT) simt_bwd_kernel(const T* __restrict__ Q, const T* __restrict__ K,
                                                      const T* __restrict__ V, const T* __restrict__ dO,
                                                      const float* __restrict__ lse, const float* __restrict__ Dv,
                                                      const float* __restrict__ bias,
                                                      const int32_t* __restrict__ expiry,
                                                      const uint32_t* __restrict__ bitmap, float* __restrict__ dQacc,
                                                      T* __restrict__ dK, T* __restrict__ dV, float* __restrict__ dM,
                                                      Prob P, int use_bitmap) {
    constexpr int LDQ = D + 1, LDS = BN + 1;
    extern __shared__ float sm[];
    float* sK = sm;                     // [BN][LDQ]
    float* sV = sK + BN * LDQ;          // [BN][LDQ]
    float* sQ = sV + BN * LDQ;          // [BM][LDQ]
    float* sG = sQ + BM * LDQ;          // dO tile [BM][LDQ]
    float* sP = sG + BM * LDQ;          // [BM][LDS]
    float* sD = sP + BM * LDS;          // dS [BM][LDS]
    float* sLse = sD + BM * LDS;        // [BM]
    float* sDv = sLse + BM;             // [BM]
    float* sB = sDv + BM;               // [BN]
    float* sdM = sB + BN;               // [BN]
    int* sE = reinterpret_cast<int*>(sdM + BN);

    const int kt = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
    const int j0 = kt * BN, L = P.L;
    const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
    load_tile(sK, LDQ, K + b * P.ks[0] + hk * P.ks[2], P.ks[1], j0, L, D);
    load_tile(sV, LDQ, V + b * P.vs[0] + hk * P.vs[2], P.vs[1], j0, L, D);

    float adk[4][D / 16], adv[4][D / 16];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < D / 16; ++c) adk[a][c] = adv[a][c] = 0.0f;

    for (int g = 0; g < P.G; ++g) {
        const int h = hk * P.G + g, bh = b * P.Hq + h;
        __syncthreads();
        if (tid < BN) {
            int j = j0 + tid;
            sB[tid] = j < L ? bias[(size_t)bh * L + j] : 0.0f;
            sE[tid] = j < L ? expiry[(size_t)bh * L + j] : 0;
            sdM[tid] = 0.0f;
        }
        for (int i0 = P.causal ? (j0 / BM) * BM : 0; i0 < L; i0 += BM) {
            if (use_bitmap && !bitmap_test(bitmap, P.Tr, P.Wd, bh, i0 / P.bm, j0 / P.bn)) continue;
            __syncthreads();
            load_tile(sQ, LDQ, Q + b * P.qs[0] + h * P.qs[2], P.qs[1], i0, L, D);
            load_tile(sG, LDQ, dO + b * P.os[0] + h * P.os[2], P.os[1], i0, L, D);
            if (tid < BM) {
                int i = i0 + tid;
                sLse[tid] = i < L ? lse[(size_t)bh * L + i] : 0.0f;
                sDv[tid] = i < L ? Dv[(size_t)bh * L + i] : 0.0f;
            }
            __syncthreads();
            float s[4][4], dp[4][4];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int c = 0; c < 4; ++c) s[a][c] = dp[a][c] = 0.0f;
            for (int kk = 0; kk < D; ++kk) {
                float qa[4], ga[4], kb[4], vb[4];
#pragma unroll
                for (int a = 0; a < 4; ++a) { qa[a] = sQ[(ty + 16 * a) * LDQ + kk]; ga[a] = sG[(ty + 16 * a) * LDQ + kk]; }
#pragma unroll
                for (int c = 0; c < 4; ++c) { kb[c] = sK[(tx + 16 * c) * LDQ + kk]; vb[c] = sV[(tx + 16 * c) * LDQ + kk]; }
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        s[a][c] = fmaf(qa[a], kb[c], s[a][c]);
                        dp[a][c] = fmaf(ga[a], vb[c], dp[a][c]);
                    }
            }
            float colsum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    int r = ty + 16 * a, cc = tx + 16 * c, i = i0 + r, j = j0 + cc;
                    bool ok = (j <= i || !P.causal) && i < sE[cc] && i < L;
                    float p = ok ? __expf(s[a][c] * P.scale + sB[cc] - sLse[r]) : 0.0f;
                    float ds = p * (dp[a][c] - sDv[r]);
                    sP[r * LDS + cc] = p;
                    sD[r * LDS + cc] = ds;
                    colsum[c] += ds;
                }
#pragma unroll
            for (int c = 0; c < 4; ++c) atomicAdd(&sdM[tx + 16 * c], colsum[c]);
            __syncthreads();
            // dV_j += P^T dO_i ; dK_j += dS^T Q_i   (rows of the output = keys ty+16a, columns tx+16c)
            for (int i = 0; i < BM; ++i) {
                float pa[4], da[4];
#pragma unroll
                for (int a = 0; a < 4; ++a) { pa[a] = sP[i * LDS + ty + 16 * a]; da[a] = sD[i * LDS + ty + 16 * a]; }
#pragma unroll
                for (int c = 0; c < D / 16; ++c) {
                    float gg = sG[i * LDQ + tx + 16 * c], qq = sQ[i * LDQ + tx + 16 * c];
#pragma unroll
                    for (int a = 0; a < 4; ++a) {
                        adv[a][c] = fmaf(pa[a], gg, adv[a][c]);
                        adk[a][c] = fmaf(da[a], qq, adk[a][c]);
                    }
                }
            }
            // dQ_i += dS K_j * scale
            float adq[4][D / 16];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int c = 0; c < D / 16; ++c) adq[a][c] = 0.0f;
            for (int j = 0; j < BN; ++j) {
                float da[4];
#pragma unroll
                for (int a = 0; a < 4; ++a) da[a] = sD[(ty + 16 * a) * LDS + j];
#pragma unroll
                for (int c = 0; c < D / 16; ++c) {
                    float kk = sK[j * LDQ + tx + 16 * c];
#pragma unroll
                    for (int a = 0; a < 4; ++a) adq[a][c] = fmaf(da[a], kk, adq[a][c]);
                }
            }
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                int i = i0 + ty + 16 * a;
                if (i >= L) continue;
                float* dq = dQacc + (((size_t)b * L + i) * P.Hq + h) * D;
#pragma unroll
                for (int c = 0; c < D / 16; ++c) atomicAdd(dq + tx + 16 * c, adq[a][c] * P.scale);
            }
        }
        __syncthreads();
        if (tid < BN && j0 + tid < L) dM[(size_t)bh * L + j0 + tid] = sdM[tid];
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        int j = j0 + ty + 16 * a;
        if (j >= L) continue;
        T* dk = dK + b * P.ks[0] + (int64_t)j * P.ks[1] + hk * P.ks[2];
        T* dv = dV + b * P.vs[0] + (int64_t)j * P.vs[1] + hk * P.vs[2];
#pragma unroll
        for (int c = 0; c < D / 16; ++c) {
            store_as(dk + tx + 16 * c, adk[a][c] * P.scale);
            store_as(dv + tx + 16 * c, adv[a][c]);
        }
    }
}

// dQ accumulator [B,L,Hq,d] fp32 contiguous -> dQ in the caller's layout and type
template <typename T>
__global__ void dq_convert_kernel(const float* __restrict__ acc, T* __restrict__ dQ, Prob P) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    size_t n = (size_t)P.B * P.L * P.Hq * P.d;
    if (idx >= n) return;
    int c = idx % P.d, h = (idx / P.d) % P.Hq, i = (idx / ((size_t)P.d * P.Hq)) % P.L, b = idx / ((size_t)P.d * P.Hq * P.L);
    store_as(dQ + b * P.qs[0] + (int64_t)i * P.qs[1] + h * P.qs[2] + c, acc[idx]);
}

template <typename T, int D>
int fwd_t(const Prob& P, const void* Q, const void* K, const void* V, const float* bias, const int32_t* expiry,
          const uint32_t* bitmap, void* O, float* lse, cudaStream_t st) {
    size_t smem = (size_t)(2 * BM * (D + 1) + BN * D + BM * (BN + 1) + 3 * BM + 2 * BN) * sizeof(float);
    auto kern = simt_fwd_kernel<T, D>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DMA_ERR_CUDA;
    // a chunk of query rows that does not start on a bitmap row boundary (or comes without a bitmap) visits every key tile
    int use_bitmap = bitmap && !(P.flags & DMA_FLAG_IGNORE_BITMAP) && P.bm % BM == 0 && P.bn % BN == 0 && P.q_off % BM == 0;
    timing_mark(0, false, st);
    kern<<<dim3((P.Lq + BM - 1) / BM, P.Hq, P.B), NT, smem, st>>>((const T*)Q, (const T*)K, (const T*)V, bias, expiry,
                                                                  bitmap, (T*)O, lse, P, use_bitmap);
    timing_mark(0, true, st);
    count_launch();
    return check_launch();
}

template <typename T, int D>
int bwd_t(const Prob& P, const void* Q, const void* K, const void* V, const void* O, const void* dO, const float* lse,
          const float* bias, const int32_t* expiry, const uint32_t* bitmap, void* dQ, void* dK, void* dV, float* dM,
          void* ws, cudaStream_t st) {
    const size_t rows = (size_t)P.B * P.Hq * P.L, nq = rows * P.d;
    float* Dv = reinterpret_cast<float*>((char*)ws + kWsHeaderBytes);
    float* acc = Dv + ((rows + 63) / 64) * 64;
    rowdot_kernel<T><<<(unsigned)((rows + 7) / 8), 256, 0, st>>>((const T*)O, (const T*)dO, Dv, P);
    if (cudaMemsetAsync(acc, 0, nq * sizeof(float), st) != cudaSuccess) return DMA_ERR_CUDA;
    size_t smem = (size_t)(4 * BM * (D + 1) + 2 * BM * (BN + 1) + 2 * BM + 3 * BN) * sizeof(float);
    auto kern = simt_bwd_kernel<T, D>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DMA_ERR_CUDA;
    int use_bitmap = !(P.flags & DMA_FLAG_IGNORE_BITMAP) && P.bm % BM == 0 && P.bn % BN == 0;
    timing_mark(1, false, st);
    kern<<<dim3((P.L + BN - 1) / BN, P.Hkv, P.B), NT, smem, st>>>((const T*)Q, (const T*)K, (const T*)V, (const T*)dO,
                                                                  lse, Dv, bias, expiry, bitmap, acc, (T*)dK, (T*)dV,
                                                                  dM, P, use_bitmap);
    timing_mark(1, true, st);
    dq_convert_kernel<T><<<(unsigned)((nq + 255) / 256), 256, 0, st>>>(acc, (T*)dQ, P);
    count_launch(3);
    return check_launch();
}

}  // namespace

size_t simt_bwd_ws_bytes(const Prob& P) {
    const size_t rows = (size_t)P.B * P.Hq * P.L;
    return kWsHeaderBytes + (((rows + 63) / 64) * 64 + rows * P.d) * sizeof(float);
}

int launch_simt_fwd(const Prob& P, const void* Q, const void* K, const void* V, const float* bias,
                    const int32_t* expiry, const uint32_t* bitmap, void* O, float* lse, cudaStream_t st) {
    if (P.dtype == DMA_FP32)
        return P.d == 128 ? fwd_t<float, 128>(P, Q, K, V, bias, expiry, bitmap, O, lse, st)
                          : fwd_t<float, 64>(P, Q, K, V, bias, expiry, bitmap, O, lse, st);
    return P.d == 128 ? fwd_t<__nv_bfloat16, 128>(P, Q, K, V, bias, expiry, bitmap, O, lse, st)
                      : fwd_t<__nv_bfloat16, 64>(P, Q, K, V, bias, expiry, bitmap, O, lse, st);
}

int launch_simt_bwd(const Prob& P, const void* Q, const void* K, const void* V, const void* O, const void* dO,
                    const float* lse, const float* bias, const int32_t* expiry, const uint32_t* bitmap, void* dQ,
                    void* dK, void* dV, float* dM, void* ws, cudaStream_t st) {
#define DMA_BWD_ARGS P, Q, K, V, O, dO, lse, bias, expiry, bitmap, dQ, dK, dV, dM, ws, st
    if (P.dtype == DMA_FP32) return P.d == 128 ? bwd_t<float, 128>(DMA_BWD_ARGS) : bwd_t<float, 64>(DMA_BWD_ARGS);
    return P.d == 128 ? bwd_t<__nv_bfloat16, 128>(DMA_BWD_ARGS) : bwd_t<__nv_bfloat16, 64>(DMA_BWD_ARGS);
#undef DMA_BWD_ARGS
}

}  // namespace dma
