// Tensor-core forward (Sec. 4.2, Alg. 1) for bf16, d = 128, on sm_100a: TMA-staged Q/K/V tiles, tcgen05 MMAs with
// accumulators in tensor memory, online softmax in registers, bitmap-driven tile skipping.
//
// One CTA owns two consecutive 128-row query tiles of one (batch, head) and walks the union of their active key
// tiles. Warp roles (12 warps):
//   warps 0-3 / 4-7  softmax group 0 / 1: thread r owns query row r of its tile (TMEM lane r): reads S, adds the
//                    bias, applies the validity test j <= i < expiry[j], keeps the running max / sum, writes P (bf16)
//                    back to tensor memory over S, rescales O when the max has grown, and finally normalises O
//   warp 8           producer: builds the tile schedule from the bitmap, then issues the TMA loads of K and V per
//                    active key tile (inactive tiles are never loaded); warp 10 stages bias / expiry vectors
//   warp 9           MMA issuer: S_w = Q_w K^T, O_w += P_w V, ping-ponging between the two query tiles so that the
//                    tensor cores run one tile's GEMMs while the other tile's softmax is in flight
// Tensor memory (512 columns): S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512); P_w aliases columns [0,64) of S_w.
// The log-sum-exp replaces Alg. 1's (l, m) pair. Scores are kept in the log2 domain: x = log2(e) (s scale + bias).
#include <type_traits>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace dma {
namespace {

using namespace ptx;

constexpr int kStages = 2;
constexpr int kMaxSched = 1024;               // key tiles per CTA schedule (L <= 131072)
constexpr int kThreads = 384;
constexpr uint32_t kTileBytes = 128 * 128 * 2;   // one 128 x 128 bf16 tile = two 16 KB swizzled half tiles
constexpr float kRescaleThreshold = 8.0f;     // log2 units: P stays below 2^8, O is rescaled only on larger jumps

struct SharedStorage {
    alignas(1024) uint8_t q[2][kTileBytes];
    alignas(1024) uint8_t k[kStages][kTileBytes];
    alignas(1024) uint8_t v[kStages][kTileBytes];
    alignas(16) float bias[kStages][128];     // log2(e) * bias of the staged key tile
    alignas(16) int len[kStages][128];        // expiry[j] (0 beyond L): row i keeps key j iff j <= i < expiry[j]
    uint32_t sched[kMaxSched];                // key tile | use by tile 0 << 30 | use by tile 1 << 31
    uint64_t q_full, k_full[kStages], v_full[kStages], k_empty[kStages], v_empty[kStages];
    uint64_t s_full[2], p_ready[2], o_done[2];
    uint32_t tmem_base;
    int n_iters;
    int abort_flag;
};

struct FwdParams {
    const float* bias;
    const int32_t* expiry;
    const uint32_t* bitmap;
    __nv_bfloat16* O;
    float* lse;
    int32_t* status;
    int B, Hq, G, L, Tr, Tc, Wd, ignore_bitmap;
    float scale_log2;                          // softmax scale * log2(e)
    int64_t os_b, os_l, os_h;
};

__device__ __forceinline__ uint32_t use_bit(uint32_t entry, int w) { return (entry >> (30 + w)) & 1u; }

__global__ void __launch_bounds__(kThreads, 1)
fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
           const __grid_constant__ CUtensorMap tmV, const FwdParams P) {
    extern __shared__ uint8_t smem_raw[];
    SharedStorage& S = *reinterpret_cast<SharedStorage*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x, b = bh / P.Hq, h = bh % P.Hq, hk = h / P.G;
    const int npairs = (P.Tr + 1) / 2;
    const int pair = npairs - 1 - (int)blockIdx.y;          // heaviest query tiles first
    const int qt0 = 2 * pair, qt1 = 2 * pair + 1;
    const bool has1 = qt1 < P.Tr;
    volatile int* abort_flag = &S.abort_flag;

    if (tid == 0) {
        mbar_init(&S.q_full, 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&S.k_full[s], 2);      // TMA bytes of K + the staged bias / expiry vectors
            mbar_init(&S.v_full[s], 1);
            mbar_init(&S.k_empty[s], 1);
            mbar_init(&S.v_empty[s], 1);
        }
        for (int w = 0; w < 2; ++w) {
            mbar_init(&S.s_full[w], 1);
            mbar_init(&S.p_ready[w], 128);
            mbar_init(&S.o_done[w], 1);
        }
        S.abort_flag = 0;
        S.n_iters = 0;
        fence_barrier_init();
    }
    if (warp == 9) {
        tmem_alloc(&S.tmem_base, 512);
        tmem_relinquish();
    }
    if (warp == 8) {
        // schedule: ascending key tiles that at least one of the two query tiles uses
        if (lane == 0) { prefetch_tmap(&tmQ); prefetch_tmap(&tmK); prefetch_tmap(&tmV); }
        const int kt_last = min(has1 ? qt1 : qt0, P.Tc - 1);
        int n = 0;
        for (int base = 0; base <= kt_last; base += 32) {
            const int kt = base + lane;
            uint32_t u0 = 0, u1 = 0;
            if (kt <= kt_last) {
                u0 = kt <= qt0 && (P.ignore_bitmap || bitmap_test(P.bitmap, P.Tr, P.Wd, bh, qt0, kt));
                u1 = has1 && kt <= qt1 && (P.ignore_bitmap || bitmap_test(P.bitmap, P.Tr, P.Wd, bh, qt1, kt));
            }
            const uint32_t act = __ballot_sync(0xffffffffu, u0 | u1);
            if (u0 | u1) S.sched[n + __popc(act & ((1u << lane) - 1))] = (uint32_t)kt | (u0 << 30) | (u1 << 31);
            n += __popc(act);
        }
        if (lane == 0) S.n_iters = n;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = S.tmem_base;
    const int n_iters = S.n_iters;

    if (warp < 8) {
        // =========================================== softmax groups ===========================================
        setmaxnreg_inc<216>();
        const int w = warp >> 2;
        const int r = tid & 127;
        const int qt = w ? qt1 : qt0;
        const int i = qt * 128 + r;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_base + w * 128;
        const uint32_t tO = tmem + lane_base + 256 + w * 128;
        float m_ref = -INFINITY, l = 0.0f;
        int n_used = 0;
        bool ok = true;
        for (int it = 0; it < n_iters && ok; ++it) {
            const uint32_t entry = S.sched[it];
            if (!use_bit(entry, w)) continue;
            const int st = it % kStages, j0 = (int)(entry & 0xFFFFF) * 128;
            ok = mbar_wait_warp(&S.s_full[w], n_used & 1, abort_flag) && mbar_wait_warp(&S.k_full[st], (it / kStages) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            float x[128];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t raw[32];
                tmem_ld32(tS + c * 32, raw);
                tc_wait_ld();
#pragma unroll
                for (int u = 0; u < 32; ++u) x[c * 32 + u] = __uint_as_float(raw[u]);
            }
            // x = log2e (s scale + bias) where row i keeps key j (j <= i < expiry[j]), else -inf. Off the diagonal
            // j <= i always holds and one compare against the staged expiry decides; the two cases are separate
            // loops so that neither pays for the other's test. Four independent max chains.
            float mxa[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            auto score_pass = [&](auto diag) {
                constexpr bool kDiag = decltype(diag)::value;
#pragma unroll
                for (int c = 0; c < 128; c += 4) {
                    const float4 bb = *reinterpret_cast<const float4*>(&S.bias[st][c]);
                    const int4 ee = *reinterpret_cast<const int4*>(&S.len[st][c]);
                    const float bv[4] = {bb.x, bb.y, bb.z, bb.w};
                    const int ev[4] = {ee.x, ee.y, ee.z, ee.w};
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float xv = fmaf(x[c + u], P.scale_log2, bv[u]);
                        const bool valid = kDiag ? (j0 + c + u <= i && i < ev[u]) : (i < ev[u]);
                        x[c + u] = valid ? xv : -INFINITY;
                        mxa[u] = fmaxf(mxa[u], x[c + u]);
                    }
                }
            };
            if (j0 + 127 > qt * 128) score_pass(std::true_type{}); else score_pass(std::false_type{});
            const float mx = fmaxf(fmaxf(mxa[0], mxa[1]), fmaxf(mxa[2], mxa[3]));
            const float m_new = fmaxf(m_ref, mx);
            if (n_used == 0) {
                m_ref = m_new;
            } else if (__any_sync(0xffffffffu, m_new > m_ref + kRescaleThreshold)) {
                // O_w *= 2^(m_ref - m_new): the previous P V product must have landed first
                ok = mbar_wait_warp(&S.o_done[w], (n_used - 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const float f = (m_new == -INFINITY) ? 1.0f : ex2(m_ref - m_new);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tO + c * 32, o);
                    tc_wait_ld();
#pragma unroll
                    for (int u = 0; u < 32; ++u) o[u] = __float_as_uint(__uint_as_float(o[u]) * f);
                    tmem_st32(tO + c * 32, o);
                }
                tc_wait_st();
                l *= f;
                m_ref = m_new;
            }
            const float m_use = (m_ref == -INFINITY) ? 0.0f : m_ref;
            float sa[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t pk[32];
#pragma unroll
                for (int c = 0; c < 64; c += 2) {
                    const float p0 = ex2(x[half * 64 + c] - m_use), p1 = ex2(x[half * 64 + c + 1] - m_use);
                    sa[(c >> 1) & 3] += p0 + p1;
                    pk[c >> 1] = pack_bf16(p0, p1);
                }
                tmem_st32(tS + half * 32, pk);
            }
            l += (sa[0] + sa[1]) + (sa[2] + sa[3]);
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(&S.p_ready[w]);
            ++n_used;
        }
        // epilogue: O_w / l -> bf16 rows, log-sum-exp in natural log
        const bool exists = w == 0 || has1;
        if (ok && exists && n_used > 0) ok = mbar_wait_warp(&S.o_done[w], (n_used - 1) & 1, abort_flag);
        if (ok && exists) {
            tc_fence_after();
            const float inv = l > 0.0f ? 1.0f / l : 0.0f;
            __nv_bfloat16* orow = P.O + b * P.os_b + (int64_t)i * P.os_l + h * P.os_h;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t o[32];
                if (n_used > 0) {
                    tmem_ld32(tO + c * 32, o);
                    tc_wait_ld();
                } else {
#pragma unroll
                    for (int u = 0; u < 32; ++u) o[u] = 0;
                }
                if (i < P.L) {
#pragma unroll
                    for (int u = 0; u < 32; u += 8) {
                        uint4 pkt;
                        pkt.x = pack_bf16(__uint_as_float(o[u]) * inv, __uint_as_float(o[u + 1]) * inv);
                        pkt.y = pack_bf16(__uint_as_float(o[u + 2]) * inv, __uint_as_float(o[u + 3]) * inv);
                        pkt.z = pack_bf16(__uint_as_float(o[u + 4]) * inv, __uint_as_float(o[u + 5]) * inv);
                        pkt.w = pack_bf16(__uint_as_float(o[u + 6]) * inv, __uint_as_float(o[u + 7]) * inv);
                        *reinterpret_cast<uint4*>(orow + c * 32 + u) = pkt;
                    }
                }
            }
            if (i < P.L) P.lse[(size_t)bh * P.L + i] = l > 0.0f ? 0.6931471805599453f * (m_ref + log2f(l)) : -INFINITY;
        }
    } else {
        setmaxnreg_dec<72>();   // 4 warps x 96 registers released = 8 warps x 48 acquired below
        if (warp == 8) {
            // =========================================== producer ===========================================
            if (lane == 0) {
                mbar_arrive_expect_tx(&S.q_full, has1 ? 2 * kTileBytes : kTileBytes);
                for (int w = 0; w < (has1 ? 2 : 1); ++w)
                    for (int hf = 0; hf < 2; ++hf)
                        tma_load_4d(&S.q[w][hf * (kTileBytes / 2)], &tmQ, &S.q_full, hf * 64, (qt0 + w) * 128, h, b);
            }
            // K and V of a stage are released separately (K once its S = Q K^T products are done, V after P V), so
            // the next K tile is in flight about two key tiles ahead of its use
            bool ok = true;
            for (int it = 0; it < n_iters && ok; ++it) {
                const int st = it % kStages, j0 = (int)(S.sched[it] & 0xFFFFF) * 128;
                if (it >= kStages) ok = mbar_wait_warp(&S.k_empty[st], ((it / kStages) - 1) & 1, abort_flag);
                if (!ok) break;
                if (lane == 0) {
                    mbar_arrive_expect_tx(&S.k_full[st], kTileBytes);
                    tma_load_4d(&S.k[st][0], &tmK, &S.k_full[st], 0, j0, hk, b);
                    tma_load_4d(&S.k[st][kTileBytes / 2], &tmK, &S.k_full[st], 64, j0, hk, b);
                }
                if (it >= kStages) ok = mbar_wait_warp(&S.v_empty[st], ((it / kStages) - 1) & 1, abort_flag);
                if (!ok) break;
                if (lane == 0) {
                    mbar_arrive_expect_tx(&S.v_full[st], kTileBytes);
                    tma_load_4d(&S.v[st][0], &tmV, &S.v_full[st], 0, j0, hk, b);
                    tma_load_4d(&S.v[st][kTileBytes / 2], &tmV, &S.v_full[st], 64, j0, hk, b);
                }
            }
            // tail: the last stages' release arrivals must land before the CTA's shared memory is given up
            for (int it = max(0, n_iters - kStages); it < n_iters && ok; ++it)
                ok = mbar_wait_warp(&S.k_empty[it % kStages], (it / kStages) & 1, abort_flag) &&
                     mbar_wait_warp(&S.v_empty[it % kStages], (it / kStages) & 1, abort_flag);
        } else if (warp == 10) {
            // =========================================== stager ===========================================
            // bias (log2 domain) and expiry of each key tile -> shared memory; the global loads run one tile ahead
            auto fetch = [&](int it, float (&bv)[4], int (&ev)[4]) {
                const int j0 = (int)(S.sched[it] & 0xFFFFF) * 128;
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const int j = j0 + lane + 32 * t;
                    bv[t] = j < P.L ? P.bias[(size_t)bh * P.L + j] : 0.0f;
                    ev[t] = j < P.L ? P.expiry[(size_t)bh * P.L + j] : 0;
                }
            };
            float bv[4] = {0.f, 0.f, 0.f, 0.f};
            int ev[4] = {0, 0, 0, 0};
            if (n_iters > 0) fetch(0, bv, ev);
            bool ok = true;
            for (int it = 0; it < n_iters && ok; ++it) {
                const int st = it % kStages;
                float bn[4] = {0.f, 0.f, 0.f, 0.f};
                int en[4] = {0, 0, 0, 0};
                if (it + 1 < n_iters) fetch(it + 1, bn, en);
                // the vectors of this stage were last read by the softmax groups before they released P (hence before P V)
                if (it >= kStages) ok = mbar_wait_warp(&S.v_empty[st], ((it / kStages) - 1) & 1, abort_flag);
                if (!ok) break;
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    S.bias[st][lane + 32 * t] = bv[t] * 1.4426950408889634f;
                    S.len[st][lane + 32 * t] = ev[t];
                    bv[t] = bn[t];
                    ev[t] = en[t];
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&S.k_full[st]);
            }
        } else if (warp == 9 && lane == 0) {
            // =========================================== MMA issuer ===========================================
            constexpr uint32_t idesc_s = idesc_bf16(128, 128, 0, 0);     // Q (K-major) x K (K-major)
            constexpr uint32_t idesc_pv = idesc_bf16(128, 128, 0, 1);    // P (TMEM)    x V (MN-major)
            auto issue_s = [&](int w, int st) {
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t off = (kk >> 2) * (kTileBytes / 2) + (kk & 3) * 32;
                    mma_ss(tmem + w * 128, smem_desc_sw128(smem_u32(&S.q[w][off]), 16, 1024),
                           smem_desc_sw128(smem_u32(&S.k[st][off]), 16, 1024), idesc_s, kk > 0);
                }
                tc_commit(&S.s_full[w]);
            };
            int n_p[2] = {0, 0};
            bool ok = mbar_wait(&S.q_full, 0, abort_flag);
            if (ok && n_iters > 0) {
                ok = mbar_wait(&S.k_full[0], 0, abort_flag);
                if (ok) {
                    tc_fence_after();
                    for (int w = 0; w < 2; ++w)
                        if (use_bit(S.sched[0], w)) issue_s(w, 0);
                    tc_commit(&S.k_empty[0]);
                }
            }
            for (int it = 0; it < n_iters && ok; ++it) {
                const int st = it % kStages, nst = (it + 1) % kStages;
                const uint32_t entry = S.sched[it], next = it + 1 < n_iters ? S.sched[it + 1] : 0u;
                ok = mbar_wait(&S.v_full[st], (it / kStages) & 1, abort_flag);
                bool k_ready = false;
                for (int w = 0; w < 2 && ok; ++w) {
                    if (use_bit(entry, w)) {
                        ok = mbar_wait(&S.p_ready[w], n_p[w] & 1, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk)
                            mma_ts(tmem + 256 + w * 128, tmem + w * 128 + kk * 8,
                                   smem_desc_sw128(smem_u32(&S.v[st][kk * 2048]), kTileBytes / 2, 1024), idesc_pv,
                                   (n_p[w] > 0 || kk > 0) ? 1u : 0u);
                        tc_commit(&S.o_done[w]);
                        ++n_p[w];
                    }
                    if (use_bit(next, w)) {
                        if (!k_ready) {
                            ok = mbar_wait(&S.k_full[nst], ((it + 1) / kStages) & 1, abort_flag);
                            if (!ok) break;
                            tc_fence_after();
                            k_ready = true;
                        }
                        issue_s(w, nst);
                    }
                }
                if (ok) {
                    tc_commit(&S.v_empty[st]);
                    if (it + 1 < n_iters) tc_commit(&S.k_empty[nst]);
                }
            }
        }
    }
    // teardown: every role falls through to here, also after a timed-out wait
    tc_fence_before();
    __syncthreads();
    if (warp == 9) {
        tc_fence_after();
        tmem_dealloc(tmem, 512);
    }
    if (tid == 0 && S.abort_flag) atomicExch(P.status, (int32_t)DMA_ERR_DEVICE_TIMEOUT);
}

}  // namespace

EncodeTiledFn get_encode_tiled() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

int make_tmap_bf16(CUtensorMap* m, const void* base, int B, int L, int H, int d, const int64_t strides[3], int rows) {
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return DMA_ERR_CUDA;
    cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)L, (cuuint64_t)H, (cuuint64_t)B};
    cuuint64_t str[3] = {(cuuint64_t)strides[1] * 2, (cuuint64_t)strides[2] * 2, (cuuint64_t)strides[0] * 2};   // bytes, dims 1..3
    cuuint32_t box[4] = {64, (cuuint32_t)rows, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, str, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DMA_OK : DMA_ERR_CUDA;
}

int make_tmap_f32_rows(CUtensorMap* m, const void* base, int B, int L, int H, int rows, int channels) {
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return DMA_ERR_CUDA;
    cuuint64_t dims[4] = {128, (cuuint64_t)H, (cuuint64_t)L, (cuuint64_t)B};
    cuuint64_t str[3] = {128 * 4, (cuuint64_t)H * 128 * 4, (cuuint64_t)L * H * 128 * 4};
    cuuint32_t box[4] = {(cuuint32_t)channels, 1, (cuuint32_t)rows, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<void*>(base), dims, str, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DMA_OK : DMA_ERR_CUDA;
}

size_t tc_fwd_ws_bytes(const Prob&) { return kWsHeaderBytes; }

int launch_tc_fwd(const Prob& P, const void* Q, const void* K, const void* V, const float* bias,
                  const int32_t* expiry, const uint32_t* bitmap, void* O, float* lse, void* ws, cudaStream_t st) {
    if (P.Tc > kMaxSched) return DMA_ERR_UNSUPPORTED;
    CUtensorMap tmQ, tmK, tmV;
    int rc;
    if ((rc = make_tmap_bf16(&tmQ, Q, P.B, P.L, P.Hq, P.d, P.qs, 128))) return rc;
    if ((rc = make_tmap_bf16(&tmK, K, P.B, P.L, P.Hkv, P.d, P.ks, 128))) return rc;
    if ((rc = make_tmap_bf16(&tmV, V, P.B, P.L, P.Hkv, P.d, P.vs, 128))) return rc;
    FwdParams fp;
    fp.bias = bias; fp.expiry = expiry; fp.bitmap = bitmap; fp.O = (__nv_bfloat16*)O; fp.lse = lse;
    fp.status = (int32_t*)ws;
    fp.B = P.B; fp.Hq = P.Hq; fp.G = P.G; fp.L = P.L; fp.Tr = P.Tr; fp.Tc = P.Tc; fp.Wd = P.Wd;
    fp.ignore_bitmap = (P.flags & DMA_FLAG_IGNORE_BITMAP) ? 1 : 0;
    fp.scale_log2 = P.scale * 1.4426950408889634f;
    fp.os_b = P.os[0]; fp.os_l = P.os[1]; fp.os_h = P.os[2];
    const size_t smem = sizeof(SharedStorage) + 1024;
    if (cudaFuncSetAttribute(fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DMA_ERR_CUDA;
    dim3 grid(P.B * P.Hq, (P.Tr + 1) / 2);
    fwd_kernel<<<grid, kThreads, smem, st>>>(tmQ, tmK, tmV, fp);
    count_launch();
    return check_launch();
}

}  // namespace dma
