// Tensor-core forward (Sec. 4.2, Alg. 1) for bf16, d = 128 or 64, on sm_100a: TMA-staged Q/K/V tiles, tcgen05 MMAs with
// accumulators in tensor memory, online softmax in registers, bitmap-driven tile skipping.
//
// One CTA owns two consecutive 128-row query tiles of one (batch, head) and walks the union of their active key
// tiles. Bias and mask are folded into the score GEMM: S_w = Q_w K^T gets a ninth k-step whose operands the stager
// warps build per (key tile, query tile) - it adds bias / scale, -BIG for keys that expired before the tile's rows
// and a step function per key that expires inside them - so that the softmax warps read finished scores from tensor
// memory and touch no shared memory per element. Diagonal tiles, and tiles in which more than 13 keys expire inside
// the query tile's rows, take the general path with the explicit test j <= i < expiry[j].
// Warp roles (12 warps):
//   warps 4-7 / 8-11 softmax group 0 / 1: thread r owns query row r of its tile (TMEM lane r): row max, lazy rescale of
//                    O, p = 2^(x c - stab), row sum, P (bf16) written back to tensor memory over S, final normalisation
//   warp 0           producer: builds the tile schedule from the bitmap, then issues the TMA loads of K and V per
//                    active key tile (inactive tiles are never loaded); K and V stages are released separately
//   warp 1           MMA issuer (whole warp, warp-uniform values, one elected lane issues): S_w = Q_w K^T (+ ninth
//                    k-step), O_w += P_w V, ping-ponging between the two query tiles
//   warps 2, 3       stagers for query tile 0 / 1: ninth k-step operands, expiry vector, fast / general flag
// Tensor memory (512 columns): S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512); P_w aliases columns [0,64) of S_w.
// kD = 64 (its own instantiations): Q, K and V tiles are one 16 KB half tile each (the second half of every buffer stays
// unused), S = Q K^T has four k-steps and the ninth, O_w takes 64 columns.
// The log-sum-exp replaces Alg. 1's (l, m) pair.
#include <cstdlib>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace dma {
namespace {

using namespace ptx;

constexpr int kStages = 2;
constexpr int kMaxSched = 1024;               // key tiles per CTA schedule (L <= 131072)
constexpr int kThreads = 384;
constexpr int kLaunchRegs = 168;             // registers per thread the kernel must be compiled to: its setmaxnreg requests
                                            // (8 warps up by 40, 4 warps down by 80) balance only for this count, and an
                                            // unbalanced request waits forever
constexpr uint32_t kTileBytes = 128 * 128 * 2;   // one 128 x 128 bf16 tile = two 16 KB swizzled half tiles
constexpr int kMaskSlots = 13;                 // keys expiring inside a tile's rows that the ninth k-step can mask
constexpr float kSmallStab = 1048576.0f;        // 2^20: below it the stabiliser is fl(m_ref c), see the softmax groups
constexpr float kRescaleThreshold = 8.0f;     // log2 units: P stays below 2^8, O is rescaled only on larger jumps

struct SharedStorage {
    alignas(1024) uint8_t q[2][kTileBytes];
    alignas(1024) uint8_t k[kStages][kTileBytes];
    alignas(1024) uint8_t v[kStages][kTileBytes];
    // Ninth k-step of S = Q K^T, per query tile: A rows [1, 1, 1, t_0(r) .. t_12(r)], B rows [b_hi, b_mid, b_lo, -BIG [j = j_0] ..],
    // unswizzled K-major core matrices (row r, element e at (r/8) 256 + (e/8) 128 + (r%8) 16 + (e%8) 2 bytes). The
    // product adds bias / scale to the score, -BIG for keys that expired before the tile's rows, and -BIG from row
    // expiry[j_k] on for the up to 13 keys j_k that expire inside the tile's rows (t_k(r) = 1 from that row on).
    alignas(128) uint8_t aext[2][4096];
    alignas(128) uint8_t bext[2][4096];
    alignas(16) int len[kStages][128];        // expiry[j] (0 beyond L): row i keeps key j iff j <= i < expiry[j]
    alignas(16) int jidx[kStages][128];       // token-compacted mode: the key index of each gathered column
    int thr[2][16];                           // stager scratch: row thresholds of the keys that expire inside the tile
    uint32_t fast[kStages][2];                // bit 0: the extra k-step carries the whole mask of this (key tile, query tile);
                                              // token-compacted mode: bit q (0-3) = 32-column chunk q needs the per-element test;
                                              // bits 8-15: 16-key blocks that hold a key some row of the query tile may keep
    uint32_t sched[kMaxSched];                // key tile | use by tile 0 << 30 | use by tile 1 << 31
    uint64_t q_full, k_full[kStages], v_full[kStages], k_empty[kStages], v_empty[kStages];
    uint64_t s_full[2], p_half[2], p_ready[2], o_done[2];
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
    float inv_scale;                           // 1 / softmax scale
    float rescale_gap;                         // growth of a row max (score units) beyond which O is rescaled
    // token-compacted mode: per (batch, head, pair of query tiles) the list of keys that some row of the
    // pair keeps (see compact_lists_kernel), padded with -1 to a multiple of 128 (ccap entries per list), and its length
    const int* cidx;
    const int* ccnt;
    const __nv_bfloat16* Kg;                   // K and V base pointers for the row gathers (strides below)
    const __nv_bfloat16* Vg;
    int ccap, Hkv;
    int causal;                                // 0: key j is visible to every row (token-compacted mode only)
    int Lq, q_off, Trq;                        // chunk of query rows (token-compacted mode only): Q, O, lse hold rows q_off .. q_off + Lq - 1; Trq = its 128-row tiles
    int64_t os_b, os_l, os_h;
    int64_t ks_b, ks_l, ks_h, vs_b, vs_l, vs_h;
};


__device__ __forceinline__ uint32_t use_bit(uint32_t entry, int w) { return (entry >> (30 + w)) & 1u; }

// Warp roles. The four service warps come FIRST: among ready warps the schedulers favour the older (lower-numbered) ones,
// and a stager that gets an issue slot only when both softmax warps of its scheduler stall was measured to need ~3600
// cycles for the few hundred instructions of one key tile.
constexpr int kWarpProducer = 0, kWarpIssuer = 1, kWarpStager0 = 2, kWarpStager1 = 3, kFirstSoftmaxWarp = 4;

// kCompact: instead of walking the active 128-key tiles of the bitmap, the CTA walks its gathered key list (keys that
// at least one of its 256 query rows keeps, at most w + 256 of them). Warps 0 and 3 fetch the K and V rows with 16-byte
// asynchronous copies into the swizzled tile layout (TMA row gathers of four rows were measured at ~70 cycles per
// request: too slow), warp 2 builds the B rows of the ninth k-step (bias, and -BIG for columns no row of the tile keeps; the A
// rows are constant) and flags the 32-column chunks that still need the per-element test.
// kBlockSkip: MMA-block skipping inside executed tiles (DMA_FLAG_BLOCK_SKIP), a separate instantiation so that the
// default kernel carries none of its code (the kernel is sensitive to the size of its service warps' loops).
template <bool kCompact, bool kBlockSkip, int kD>
__global__ void __launch_bounds__(kThreads, 1)
fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
           const __grid_constant__ CUtensorMap tmV, const FwdParams P) {
    static_assert(kD == 128 || kD == 64, "head dimensions of the tensor-core kernels");
    constexpr int kHalves = kD / 64;                         // 64-channel (128-byte) swizzled half tiles per operand tile
    constexpr uint32_t kLoadBytes = kHalves * (kTileBytes / 2);
    extern __shared__ uint8_t smem_raw[];
    SharedStorage& S = *reinterpret_cast<SharedStorage*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);      // warp-uniform to the compiler: role branches stay uniform
    const int bh = blockIdx.x, b = bh / P.Hq, h = bh % P.Hq, hk = h / P.G;
    const int npairs = (P.Trq + 1) / 2;
    const int pair = npairs - 1 - (int)blockIdx.y;          // heaviest query tiles first
    const int qt0 = 2 * pair, qt1 = 2 * pair + 1;           // query tiles inside the chunk (the whole sequence unless P.q_off / P.Lq say otherwise)
    const bool has1 = qt1 < P.Trq;
    const int lpair = (kCompact && !P.causal) ? 0 : pair;   // non-causal: all rows of a head keep the same keys, one list serves every pair
    volatile int* abort_flag = &S.abort_flag;

    if (tid == 0) {
        mbar_init(&S.q_full, 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&S.k_full[s], kCompact ? 33 : 3);   // K: TMA bytes + the two stager warps | 32 gathering lanes + the stager warp
            mbar_init(&S.v_full[s], kCompact ? 32 : 1);
            mbar_init(&S.k_empty[s], 1);
            mbar_init(&S.v_empty[s], 1);
        }
        for (int w = 0; w < 2; ++w) {
            mbar_init(&S.s_full[w], 1);
            mbar_init(&S.p_half[w], 4);          // one arrival per softmax warp
            mbar_init(&S.p_ready[w], 4);
            mbar_init(&S.o_done[w], 1);
        }
        S.abort_flag = 0;
        S.n_iters = 0;
        fence_barrier_init();
    }
    if (warp == kWarpIssuer) {
        tmem_alloc(&S.tmem_base, 512);
        tmem_relinquish();
    }
    if (warp == kWarpProducer) {
        // schedule: ascending key tiles that at least one of the two query tiles uses
        if (lane == 0) { prefetch_tmap(&tmQ); prefetch_tmap(&tmK); prefetch_tmap(&tmV); }
        int n = 0;
        if constexpr (kCompact) {
            // every 128-key slice of the gathered list, used by both query tiles
            n = min((P.ccnt[(size_t)bh * npairs + lpair] + 127) / 128, kMaxSched);
            for (int t = lane; t < n; t += 32) S.sched[t] = (uint32_t)t | (1u << 30) | (has1 ? (1u << 31) : 0u);
        } else {
            const int kt_last = min(has1 ? qt1 : qt0, P.Tc - 1);
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
        }
        if (lane == 0) S.n_iters = n;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = S.tmem_base;
    const int n_iters = S.n_iters;

    if (warp >= kFirstSoftmaxWarp) {
        // =========================================== softmax groups ===========================================
        setmaxnreg_inc<208>();
        const int w = (warp - kFirstSoftmaxWarp) >> 2;
        const int r = tid & 127;
        const int qt = w ? qt1 : qt0;
        const int il = qt * 128 + r;                        // row inside Q, O, lse
        const int i = P.q_off + il;                         // its position in the sequence
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_base + w * 128;
        const uint32_t tO = tmem + lane_base + 256 + w * 128;
        float m_ref = -INFINITY, r_ref = 0.0f, l = 0.0f;
        int n_used = 0;
        bool ok = true;
        for (int it = 0; it < n_iters && ok; ++it) {
            const uint32_t entry = S.sched[it];
            if (!use_bit(entry, w)) continue;
            const int st = it % kStages, j0 = (int)(entry & 0xFFFFF) * 128;
            ok = mbar_wait_warp(&S.s_full[w], n_used & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            // The stagers' flag is read only now. The S product was issued after k_full[st] completed, so the flag of THIS
            // iteration is in place. (Waiting on k_full[st] here instead is wrong: a tile that skipped earlier key tiles
            // has not followed that barrier's phases, and a parity wait on a barrier it is a whole phase ahead of returns
            // at once, before the stager has written the flag.)
            const uint32_t tile_flags = S.fast[st][w];
            const bool fast_tile = kCompact || (tile_flags & 1u) != 0;      // token-compacted mode: the low bits are a chunk mask instead
            // The accumulator holds q.k + bias / scale (+ -BIG where the ninth k-step masks). On the fast path that
            // is the whole masked score; otherwise (diagonal tile, or more than 13 keys expiring inside the tile's
            // rows) the validity test j <= i < expiry[j] is applied here. x = log2e * scale * score, -inf if masked.
            float x[128];
            {
                uint32_t raw[128];                 // the four loads are in flight together, one wait
#pragma unroll
                for (int c = 0; c < 4; ++c) tmem_ld32p(tS + c * 32, &raw[c * 32]);
                tc_wait_ld();
#pragma unroll
                for (int u = 0; u < 128; ++u) x[u] = __uint_as_float(raw[u]);
            }
            float mxa[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            if constexpr (kCompact) {
                // gathered columns: bias and the keys that are gone for the whole tile are already in the score; the
                // per-element test is needed only in the 32-column chunks the stager flagged (a key expiring or
                // entering inside the tile's rows)
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    if ((tile_flags >> q) & 1u) {
#pragma unroll
                        for (int c = 32 * q; c < 32 * q + 32; c += 4) {
                            const int4 ee = *reinterpret_cast<const int4*>(&S.len[st][c]);
                            const int4 jj = *reinterpret_cast<const int4*>(&S.jidx[st][c]);
                            const int ev[4] = {ee.x, ee.y, ee.z, ee.w}, jv[4] = {jj.x, jj.y, jj.z, jj.w};
#pragma unroll
                            for (int u = 0; u < 4; ++u) x[c + u] = (jv[u] <= i && i < ev[u]) ? x[c + u] : -INFINITY;
                        }
                    }
                }
            }
            if (fast_tile) {
#pragma unroll
                for (int c = 0; c < 128; c += 4) {
                    mxa[(c >> 2) & 1] = max3(mxa[(c >> 2) & 1], x[c], x[c + 1]);
                    mxa[2 + ((c >> 2) & 1)] = max3(mxa[2 + ((c >> 2) & 1)], x[c + 2], x[c + 3]);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) mxa[u] = mxa[u] < -1e20f ? -INFINITY : mxa[u];
            } else {
#pragma unroll
                for (int c = 0; c < 128; c += 4) {
                    const int4 ee = *reinterpret_cast<const int4*>(&S.len[st][c]);
                    const int ev[4] = {ee.x, ee.y, ee.z, ee.w};
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const bool valid = j0 + c + u <= i && i < ev[u];
                        x[c + u] = valid ? x[c + u] : -INFINITY;
                        mxa[u] = fmaxf(mxa[u], x[c + u]);
                    }
                }
            }
            // The running max m_ref stays in score units and the exponent is formed as (x - m_ref) * c: the difference
            // is exact for the entries that matter, whatever the magnitude of the bias.
            const float mx = fmaxf(fmaxf(mxa[0], mxa[1]), fmaxf(mxa[2], mxa[3]));
            const float m_new = fmaxf(m_ref, mx);
            auto stab_resid = [&](float m) {           // m c - stab(m); 0 for m = -inf
                const float mm = (m == -INFINITY) ? 0.0f : m;
                const float Mm = mm * P.scale_log2;
                return fabsf(Mm) < kSmallStab ? fmaf(mm, P.scale_log2, -Mm) : 0.0f;
            };
            if (n_used == 0) {
                m_ref = m_new;
                r_ref = stab_resid(m_ref);
            } else if (__any_sync(0xffffffffu, m_new > m_ref + P.rescale_gap)) {
                // O_w *= 2^(stab(m_ref) - stab(m_new)): the previous P V product must have landed first
                ok = mbar_wait_warp(&S.o_done[w], (n_used - 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const float r_new = stab_resid(m_new);
                const float f = (m_new == -INFINITY) ? 1.0f : (m_ref == -INFINITY) ? 0.0f : ex2(fmaf(m_ref - m_new, P.scale_log2, r_new - r_ref));
#pragma unroll
                for (int c = 0; c < kD / 32; ++c) {
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
                r_ref = r_new;
            }
            // p = 2^(x c - stab(m_ref)). The stabiliser is a function of the row's m_ref alone: fl(m_ref c) while that
            // is below 2^20 in magnitude (then x c - stab is one FMA per element and fl() is off by < 0.07), else the
            // exact product m_ref c, reached by taking the exact difference x - m_ref first (bias magnitudes up to the
            // fp32 range stay safe). r_ref = m_ref c - stab(m_ref) travels with m_ref.
            const float m_use = (m_ref == -INFINITY) ? 0.0f : m_ref;
            const float M = m_use * P.scale_log2, nM = -M;
            const float resid = r_ref;
            const bool small = __all_sync(0xffffffffu, fabsf(M) < kSmallStab);
            float sa[4] = {0.f, 0.f, 0.f, 0.f};
            if (small) {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t pk[32];
#pragma unroll
                    for (int c = 0; c < 64; c += 2) {
                        const float p0 = ex2(fmaf(x[half * 64 + c], P.scale_log2, nM)), p1 = ex2(fmaf(x[half * 64 + c + 1], P.scale_log2, nM));
                        sa[(c >> 1) & 3] += p0 + p1;
                        pk[c >> 1] = pack_bf16(p0, p1);
                    }
                    tmem_st32(tS + half * 32, pk);
                    if (half == 0) {          // keys 0-63 of P are complete: their half of P V can start now
                        tc_wait_st();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&S.p_half[w]);
                    }
                }
            } else {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t pk[32];
#pragma unroll
                    for (int c = 0; c < 64; c += 2) {
                        const float p0 = ex2(fmaf(x[half * 64 + c] - m_use, P.scale_log2, resid));
                        const float p1 = ex2(fmaf(x[half * 64 + c + 1] - m_use, P.scale_log2, resid));
                        sa[(c >> 1) & 3] += p0 + p1;
                        pk[c >> 1] = pack_bf16(p0, p1);
                    }
                    tmem_st32(tS + half * 32, pk);
                    if (half == 0) {
                        tc_wait_st();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&S.p_half[w]);
                    }
                }
            }
            l += (sa[0] + sa[1]) + (sa[2] + sa[3]);
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&S.p_ready[w]);      // one arrival per warp: 128 serialised arrivals cost ~400 cycles
            ++n_used;
        }
        // epilogue: O_w / l -> bf16 rows, log-sum-exp in natural log
        const bool exists = w == 0 || has1;
        if (ok && exists && n_used > 0) ok = mbar_wait_warp(&S.o_done[w], (n_used - 1) & 1, abort_flag);
        if (ok && exists) {
            tc_fence_after();
            const float inv = l > 0.0f ? 1.0f / l : 0.0f;
            __nv_bfloat16* orow = P.O + b * P.os_b + (int64_t)il * P.os_l + h * P.os_h;
#pragma unroll
            for (int c = 0; c < kD / 32; ++c) {
                uint32_t o[32];
                if (n_used > 0) {
                    tmem_ld32(tO + c * 32, o);
                    tc_wait_ld();
                } else {
#pragma unroll
                    for (int u = 0; u < 32; ++u) o[u] = 0;
                }
                if (il < P.Lq) {
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
            if (il < P.Lq) P.lse[(size_t)bh * P.Lq + il] = l > 0.0f ? 0.6931471805599453f * ((m_ref * P.scale_log2 - r_ref) + log2f(l)) : -INFINITY;
        }
    } else {
        setmaxnreg_dec<88>();   // 4 warps x 80 registers released = 8 warps x 40 acquired above
        if (kCompact && (warp == kWarpProducer || warp == kWarpStager1)) {
            // ================================ token-compacted mode: gather warps ================================
            // Warp 0 fetches the K rows of each 128-key slice of the gathered list, warp 3 the V rows: 16-byte
            // asynchronous copies into the 128-byte-swizzled tile layout (8 lanes per 128-byte half row, 4 rows per
            // instruction; padding entries (-1) are zero-filled). Each lane's copies report to the stage's barrier.
            const bool isK = warp == kWarpProducer;
            if (isK && lane == 0) {
                mbar_arrive_expect_tx(&S.q_full, has1 ? 2 * kLoadBytes : kLoadBytes);
                for (int w = 0; w < (has1 ? 2 : 1); ++w)
                    for (int hf = 0; hf < kHalves; ++hf)
                        tma_load_4d(&S.q[w][hf * (kTileBytes / 2)], &tmQ, &S.q_full, hf * 64, (qt0 + w) * 128, h, b);
            }
            const int* list = P.cidx + ((size_t)bh * npairs + lpair) * P.ccap;
            const int64_t row_stride = isK ? P.ks_l : P.vs_l;
            const __nv_bfloat16* src = (isK ? P.Kg + b * P.ks_b + hk * P.ks_h : P.Vg + b * P.vs_b + hk * P.vs_h) + (lane & 7) * 8;
            const int rsub = lane >> 3;
            const uint32_t sw0 = (uint32_t)(((lane & 7) ^ rsub) << 4), sw1 = (uint32_t)(((lane & 7) ^ (rsub + 4)) << 4);
            int jrow[32];
            if (n_iters > 0) {
#pragma unroll
                for (int q = 0; q < 32; ++q) jrow[q] = list[4 * q + rsub];
            }
            bool ok = true;
            for (int it = 0; it < n_iters && ok; ++it) {
                const int st = it % kStages;
                uint64_t* empty = isK ? &S.k_empty[st] : &S.v_empty[st];
                uint64_t* full = isK ? &S.k_full[st] : &S.v_full[st];
                uint8_t* dst = (isK ? S.k[st] : S.v[st]) + rsub * 128;
                if (it >= kStages) ok = mbar_wait_warp(empty, ((it / kStages) - 1) & 1, abort_flag);
                if (!ok) break;
#pragma unroll
                for (int q = 0; q < 32; ++q) {
                    const int j = jrow[q];
                    const __nv_bfloat16* row = src + (int64_t)max(j, 0) * row_stride;
                    uint8_t* d = dst + q * 512 + ((q & 1) ? sw1 : sw0);          // row r = 4q + rsub, chunk c ^ (r & 7)
                    cp_async16(d, row, j >= 0 ? 16 : 0);
                    if constexpr (kD == 128) cp_async16(d + kTileBytes / 2, row + 64, j >= 0 ? 16 : 0);
                }
                cp_async_arrive(full);
                if (it + 1 < n_iters) {
#pragma unroll
                    for (int q = 0; q < 32; ++q) jrow[q] = list[(it + 1) * 128 + 4 * q + rsub];
                }
            }
            for (int it = max(0, n_iters - kStages); it < n_iters && ok; ++it)
                ok = mbar_wait_warp(isK ? &S.k_empty[it % kStages] : &S.v_empty[it % kStages], (it / kStages) & 1, abort_flag);
        } else if (kCompact && warp == kWarpStager0) {
            // ================================ token-compacted mode: stager ================================
            // Per 128-key slice and query tile: the B rows of the ninth k-step (bias / scale as three bf16 terms, or
            // -BIG for a column that no row of the tile keeps; the A rows are constant ones), the key index and expiry
            // vectors, and the mask of 32-column chunks that hold a key expiring or entering inside the tile's rows (only
            // those need the per-element test). Two dependent levels of global loads, each issued a tile ahead.
            constexpr uint32_t kOne = 0x3F80u, kNegBig = 0xF14Au;     // bf16 1.0 and about -1e30
            for (int r = lane; r < 128; r += 32) {
#pragma unroll
                for (int w = 0; w < 2; ++w) {
                    uint8_t* arow = S.aext[w] + (r >> 3) * 256 + (r & 7) * 16;
                    *reinterpret_cast<uint4*>(arow) = make_uint4(kOne | (kOne << 16), kOne, 0u, 0u);
                    *reinterpret_cast<uint4*>(arow + 128) = make_uint4(0u, 0u, 0u, 0u);
                    *reinterpret_cast<uint4*>(S.bext[w] + (r >> 3) * 256 + (r & 7) * 16 + 128) = make_uint4(0u, 0u, 0u, 0u);
                }
            }
            const int* list = P.cidx + ((size_t)bh * npairs + lpair) * P.ccap;
            auto vals = [&](const int (&jv)[4], float (&bv)[4], int (&ev)[4]) {
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    bv[t] = jv[t] >= 0 ? P.bias[(size_t)bh * P.L + jv[t]] : 0.0f;
                    ev[t] = jv[t] >= 0 ? P.expiry[(size_t)bh * P.L + jv[t]] : 0;
                }
            };
            int jv[4] = {-1, -1, -1, -1}, jn[4] = {-1, -1, -1, -1}, ev[4] = {0, 0, 0, 0};
            float bv[4] = {0.f, 0.f, 0.f, 0.f};
            if (n_iters > 0) {
#pragma unroll
                for (int t = 0; t < 4; ++t) jv[t] = list[lane + 32 * t];
                vals(jv, bv, ev);
            }
            if (n_iters > 1) {
#pragma unroll
                for (int t = 0; t < 4; ++t) jn[t] = list[128 + lane + 32 * t];
            }
            bool ok = true;
            for (int it = 0; it < n_iters && ok; ++it) {
                const int st = it % kStages;
                float bn[4] = {0.f, 0.f, 0.f, 0.f};
                int en[4] = {0, 0, 0, 0}, jnn[4] = {-1, -1, -1, -1};
                if (it + 1 < n_iters) vals(jn, bn, en);
                if (it + 2 < n_iters) {
#pragma unroll
                    for (int t = 0; t < 4; ++t) jnn[t] = list[(it + 2) * 128 + lane + 32 * t];
                }
                // rows and flags are formed in registers before the waits
                uint32_t b0[2][4], b1[4], flags[2] = {0u, 0u}, live[2] = {0u, 0u};
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const float bsc = bv[t] * P.inv_scale;
                    const __nv_bfloat16 hi = __float2bfloat16_rn(bsc);
                    const float r1 = bsc - __bfloat162float(hi);
                    const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
                    const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
                    const uint32_t w0 = (uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(mid) << 16);
                    b1[t] = (uint32_t)__bfloat16_as_ushort(lo);
#pragma unroll
                    for (int w = 0; w < 2; ++w) {
                        const int i0 = P.q_off + (w ? qt1 : qt0) * 128;
                        const int first = P.causal ? jv[t] : 0;             // first row that can see the key
                        const bool dead = jv[t] < 0 || ev[t] <= i0 || first > i0 + 127;
                        const bool mixed = !dead && (ev[t] < i0 + 128 || first > i0);
                        b0[w][t] = dead ? kNegBig : w0;
                        flags[w] |= __ballot_sync(0xffffffffu, mixed) ? (1u << t) : 0u;
                        if constexpr (kBlockSkip) {
                            const uint32_t alive = __ballot_sync(0xffffffffu, !dead);
                            live[w] |= ((alive & 0xFFFFu) ? 1u : 0u) << (2 * t) | ((alive >> 16) ? 1u : 0u) << (2 * t + 1);
                        }
                    }
                }
                // the vectors of this stage were last read by the softmax groups before they released P of tile
                // it - kStages (hence before its P V); the B rows were last read by the S products of tile it - 1
                if (it >= kStages) ok = mbar_wait_warp(&S.v_empty[st], ((it / kStages) - 1) & 1, abort_flag);
                if (ok && it >= 1) ok = mbar_wait_warp(&S.k_empty[(it - 1) % kStages], ((it - 1) / kStages) & 1, abort_flag);
                if (!ok) break;
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const int c = lane + 32 * t;
                    S.jidx[st][c] = jv[t] >= 0 ? (P.causal ? jv[t] : 0) : 0x7fffffff;  // first row of the key; padding: never <= a row index
                    S.len[st][c] = ev[t];
#pragma unroll
                    for (int w = 0; w < 2; ++w)
                        *reinterpret_cast<uint4*>(S.bext[w] + (c >> 3) * 256 + (c & 7) * 16) =
                            make_uint4(b0[w][t], b0[w][t] == kNegBig ? 0u : b1[t], 0u, 0u);
                    jv[t] = jn[t]; bv[t] = bn[t]; ev[t] = en[t]; jn[t] = jnn[t];
                }
                if (lane < 2) S.fast[st][lane] = (lane ? flags[1] : flags[0]) | ((kBlockSkip ? (lane ? live[1] : live[0]) : 0xFFu) << 8);
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(&S.k_full[st]);
            }
        } else if (warp == kWarpProducer) {
            // =========================================== producer ===========================================
            if (lane == 0) {
                mbar_arrive_expect_tx(&S.q_full, has1 ? 2 * kLoadBytes : kLoadBytes);
                for (int w = 0; w < (has1 ? 2 : 1); ++w)
                    for (int hf = 0; hf < kHalves; ++hf)
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
                    mbar_arrive_expect_tx(&S.k_full[st], kLoadBytes);
                    tma_load_4d(&S.k[st][0], &tmK, &S.k_full[st], 0, j0, hk, b);
                    if constexpr (kD == 128) tma_load_4d(&S.k[st][kTileBytes / 2], &tmK, &S.k_full[st], 64, j0, hk, b);
                }
                if (it >= kStages) ok = mbar_wait_warp(&S.v_empty[st], ((it / kStages) - 1) & 1, abort_flag);
                if (!ok) break;
                if (lane == 0) {
                    mbar_arrive_expect_tx(&S.v_full[st], kLoadBytes);
                    tma_load_4d(&S.v[st][0], &tmV, &S.v_full[st], 0, j0, hk, b);
                    if constexpr (kD == 128) tma_load_4d(&S.v[st][kTileBytes / 2], &tmV, &S.v_full[st], 64, j0, hk, b);
                }
            }
            // tail: the last stages' release arrivals must land before the CTA's shared memory is given up
            for (int it = max(0, n_iters - kStages); it < n_iters && ok; ++it)
                ok = mbar_wait_warp(&S.k_empty[it % kStages], (it / kStages) & 1, abort_flag) &&
                     mbar_wait_warp(&S.v_empty[it % kStages], (it / kStages) & 1, abort_flag);
        } else if (warp == kWarpStager0 || warp == kWarpStager1) {
            // =========================================== stagers ===========================================
            // Warp 2 + w serves query tile w: per key tile it builds the ninth k-step operands described at
            // SharedStorage (warp 2 also stages the expiry vector for the general softmax path). The global loads run
            // one tile ahead and the rows are formed in registers before the wait for the blocks to be free, so that
            // only the stores are left between the previous S product and the next one.
            const int w = warp - kWarpStager0;
            const int i0 = (w ? qt1 : qt0) * 128;
            // key indices of a tile's columns, then their bias and expiry, loaded one tile before they are needed
            auto fetch_idx = [&](int it, int (&jv)[4]) {
                const int j0 = (int)(S.sched[it] & 0xFFFFF) * 128;
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    jv[t] = j0 + lane + 32 * t;
                }
            };
            auto fetch_vals = [&](const int (&jv)[4], float (&bv)[4], int (&ev)[4]) {
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const bool real = jv[t] >= 0 && jv[t] < P.L;
                    bv[t] = real ? P.bias[(size_t)bh * P.L + jv[t]] : 0.0f;
                    ev[t] = real ? P.expiry[(size_t)bh * P.L + jv[t]] : 0;
                }
            };
            constexpr uint32_t kOne = 0x3F80u, kNegBig = 0xF14Au;     // bf16 1.0 and about -1e30
            float bv[4] = {0.f, 0.f, 0.f, 0.f};
            int ev[4] = {0, 0, 0, 0}, jv[4] = {0, 0, 0, 0}, jn[4] = {0, 0, 0, 0};
            if (n_iters > 0) { fetch_idx(0, jv); fetch_vals(jv, bv, ev); }
            if (n_iters > 1) fetch_idx(1, jn);
            bool ok = true;
            for (int it = 0; it < n_iters && ok; ++it) {
                const int st = it % kStages;
                const uint32_t entry = S.sched[it];
                const bool use = use_bit(entry, w);
                float bn[4] = {0.f, 0.f, 0.f, 0.f};
                int en[4] = {0, 0, 0, 0}, jnn[4] = {0, 0, 0, 0};
                if (it + 1 < n_iters) fetch_vals(jn, bn, en);
                if (it + 2 < n_iters) fetch_idx(it + 2, jnn);
                uint32_t b0[4], b1[4], aw[4][7];
                int hot[4];
                bool fast = false;
                uint32_t live8 = 0xFFu;
                if (use) {
                    // general path needed: the tile holds keys that enter inside the query tile's rows (the diagonal tile)
                    const bool diag = (int)(entry & 0xFFFFF) == (w ? qt1 : qt0);
                    uint32_t bal[4];
                    bool mixed[4], dead[4];
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        dead[t] = ev[t] <= i0;
                        mixed[t] = !dead[t] && ev[t] < i0 + 128;
                        bal[t] = __ballot_sync(0xffffffffu, mixed[t]);
                    }
                    if constexpr (kBlockSkip) {
                        live8 = 0u;
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            const uint32_t alive = __ballot_sync(0xffffffffu, !dead[t]);     // keys 32 t .. 32 t + 31
                            live8 |= ((alive & 0xFFFFu) ? 1u : 0u) << (2 * t) | ((alive >> 16) ? 1u : 0u) << (2 * t + 1);
                        }
                    }
                    const int cnt = __popc(bal[0]) + __popc(bal[1]) + __popc(bal[2]) + __popc(bal[3]);
                    fast = !diag && cnt <= kMaskSlots;
                    if (lane < kMaskSlots) S.thr[w][lane] = 1 << 20;
                    __syncwarp();
                    int before = 0;
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const int slot = before + __popc(bal[t] & ((1u << lane) - 1));
                        before += __popc(bal[t]);
                        hot[t] = (fast && mixed[t]) ? 3 + slot : -1;          // element that holds this key's -BIG
                        if (hot[t] >= 0) S.thr[w][slot] = ev[t] - i0;
                    }
                    __syncwarp();
                    // B rows (keys): bias / scale as three bf16 terms (24 significant bits, as many as the fp32 bias
                    // has), or -BIG for a key that is gone for the whole tile
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const float bs = bv[t] * P.inv_scale;
                        const __nv_bfloat16 hi = __float2bfloat16_rn(bs);
                        const float r1 = bs - __bfloat162float(hi);
                        const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
                        const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
                        b0[t] = dead[t] ? kNegBig : ((uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(mid) << 16));
                        b1[t] = (dead[t] ? 0u : (uint32_t)__bfloat16_as_ushort(lo)) | (hot[t] == 3 ? (kNegBig << 16) : 0u);
                    }
                    // A rows (queries): ones for the bias terms, then one step function per expiring key
                    int th[kMaskSlots];
#pragma unroll
                    for (int k = 0; k < kMaskSlots; ++k) th[k] = S.thr[w][k];
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const int r = lane + 32 * t;
                        aw[t][0] = kOne | (r >= th[0] ? (kOne << 16) : 0u);
#pragma unroll
                        for (int m = 2; m < 8; ++m)
                            aw[t][m - 1] = (r >= th[2 * m - 3] ? kOne : 0u) | (r >= th[2 * m - 2] ? (kOne << 16) : 0u);
                    }
                }
                // fast[st] / len[st] were last read by the softmax groups before they released P of tile it - kStages
                // (hence before its P V); the operand blocks were last read by the S products of tile it - 1
                if (it >= kStages) ok = mbar_wait_warp(&S.v_empty[st], ((it / kStages) - 1) & 1, abort_flag);
                if (ok && it >= 1) ok = mbar_wait_warp(&S.k_empty[(it - 1) % kStages], ((it - 1) / kStages) & 1, abort_flag);
                if (!ok) break;
                if (w == 0) {
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        S.len[st][lane + 32 * t] = ev[t];
                    }
                }
                if (use) {
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const int c = lane + 32 * t;
                        uint32_t wd[8];
                        wd[0] = b0[t];
                        wd[1] = b1[t];
#pragma unroll
                        for (int m = 2; m < 8; ++m) wd[m] = (hot[t] >> 1) == m ? (kNegBig << ((hot[t] & 1) * 16)) : 0u;
                        uint8_t* brow = S.bext[w] + (c >> 3) * 256 + (c & 7) * 16;
                        *reinterpret_cast<uint4*>(brow) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
                        *reinterpret_cast<uint4*>(brow + 128) = make_uint4(wd[4], wd[5], wd[6], wd[7]);
                        uint8_t* arow = S.aext[w] + (c >> 3) * 256 + (c & 7) * 16;
                        *reinterpret_cast<uint4*>(arow) = make_uint4(kOne | (kOne << 16), aw[t][0], aw[t][1], aw[t][2]);
                        *reinterpret_cast<uint4*>(arow + 128) = make_uint4(aw[t][3], aw[t][4], aw[t][5], aw[t][6]);
                    }
                    if (lane == 0) S.fast[st][w] = (fast ? 1u : 0u) | (live8 << 8);
                }
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    bv[t] = bn[t];
                    ev[t] = en[t];
                    jv[t] = jn[t];
                    jn[t] = jnn[t];
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(&S.k_full[st]);
            }
        } else if (warp == kWarpIssuer) {
            // =========================================== MMA issuer ===========================================
            // The whole warp walks the schedule with warp-uniform values (descriptors, stage and tile indices stay in
            // the uniform datapath); one elected lane issues the tcgen05 instructions.
            constexpr uint32_t idesc_s = idesc_bf16(128, 128, 0, 0);     // Q (K-major) x K (K-major)
            constexpr uint32_t idesc_pv = idesc_bf16(128, kD, 0, 1);     // P (TMEM)    x V (MN-major)
            // operand descriptors are formed once; a stage, query tile or k-step only moves the 16-byte address field
            const uint64_t dQ0 = smem_desc_sw128(smem_u32(S.q[0]), 16, 1024), dK0 = smem_desc_sw128(smem_u32(S.k[0]), 16, 1024);
            const uint64_t dV0 = smem_desc_sw128(smem_u32(S.v[0]), kTileBytes / 2, 1024);
            const uint64_t dA0 = smem_desc_plain(smem_u32(S.aext[0]), 128, 256), dB0 = smem_desc_plain(smem_u32(S.bext[0]), 128, 256);
            const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem, 0);
            const int n_iters_u = __shfl_sync(0xffffffffu, n_iters, 0);
            // MMA-block skipping (the finer granularity inside an active tile): the stager marks the 16-key blocks of the key
            // tile in which some key may be kept by the query tile's rows, and P V multiplies the marked blocks only (P is
            // exactly zero in the others, so the result does not change). The S product is always multiplied in full: leaving
            // out a dead 64-key half was built and measured (the issuer then needs the marks BEFORE the issue, a shared-memory
            // load on the critical path: 1.98 -> 2.55 ms at L = 16384), so it stayed out.
            uint32_t live[2] = {0xFFu, 0xFFu};          // marks of the key tile whose S product was issued last, per query tile
            bool o_started[2] = {false, false};         // the O accumulator has been written (first product: no accumulate)
            auto issue_s = [&](int w, int st) {
                const uint64_t dq = dQ0 + (uint64_t)(w * (kTileBytes >> 4)), dk = dK0 + (uint64_t)(st * (kTileBytes >> 4));
                const uint32_t d_tmem = tmem_u + w * 128;
                if (elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < kD / 16; ++kk) {
                        const uint32_t off = ((kk >> 2) * (kTileBytes / 2) + (kk & 3) * 32) >> 4;
                        mma_ss(d_tmem, dq + off, dk + off, idesc_s, kk > 0);
                    }
                    mma_ss(d_tmem, dA0 + (uint64_t)(w * (4096 >> 4)), dB0 + (uint64_t)(w * (4096 >> 4)), idesc_s, 1u);
                    tc_commit(&S.s_full[w]);
                }
                __syncwarp();
                // the block marks of this key tile, for its P V product later on: read AFTER the issue (a shared-memory load
                // costs hundreds of cycles while the MMAs stream their operands, and the S products are on the critical path)
                if constexpr (kBlockSkip) live[w] = *reinterpret_cast<volatile uint32_t*>(&S.fast[st][w]) >> 8;     // (every lane reads the same word; first used at the P V issue)
            };
            int n_p[2] = {0, 0};
            bool ok = mbar_wait_warp(&S.q_full, 0, abort_flag);
            if (ok && n_iters_u > 0) {
                ok = mbar_wait_warp(&S.k_full[0], 0, abort_flag);
                if (ok) {
                    if constexpr (kCompact) fence_proxy_async();
                    tc_fence_after();
                    const uint32_t e0 = __shfl_sync(0xffffffffu, S.sched[0], 0);
#pragma unroll
                    for (int w = 0; w < 2; ++w)
                        if (use_bit(e0, w)) issue_s(w, 0);
                    if (elect_one()) tc_commit(&S.k_empty[0]);
                    __syncwarp();
                }
            }
            for (int it = 0; it < n_iters_u && ok; ++it) {
                const int st = it % kStages, nst = (it + 1) % kStages;
                const uint32_t entry = __shfl_sync(0xffffffffu, S.sched[it], 0);
                const uint32_t next = it + 1 < n_iters_u ? __shfl_sync(0xffffffffu, S.sched[it + 1], 0) : 0u;
                ok = mbar_wait_warp(&S.v_full[st], (it / kStages) & 1, abort_flag);
                if constexpr (kCompact) fence_proxy_async();     // the gathered tiles were written through the generic proxy
                bool k_ready = false;
#pragma unroll
                for (int w = 0; w < 2; ++w) {          // unrolled: n_p[] stays in registers
                    if (ok && use_bit(entry, w)) {
                        // P V in two halves of 64 keys: the first runs while the softmax group still forms the second
                        const uint64_t dv = dV0 + (uint64_t)(st * (kTileBytes >> 4));
                        const uint32_t d_tmem = tmem_u + 256 + w * 128, a_tmem = tmem_u + w * 128;
                        // blocks to multiply; an accumulator that has never been written takes block 0 in any case (P is zero there)
                        const uint32_t l8 = !kBlockSkip ? 0xFFu : (!o_started[w] && live[w] == 0u) ? 1u : live[w];
                        const uint32_t acc0 = o_started[w] ? 1u : 0u;
                        ok = mbar_wait_warp(&S.p_half[w], n_p[w] & 1, abort_flag);
                        if (ok) {
                            tc_fence_after();
                            if (elect_one()) {
                                if (l8 == 0xFFu) {                                   // the common case: every block
#pragma unroll
                                    for (int kk = 0; kk < 4; ++kk)
                                        mma_ts(d_tmem, a_tmem + kk * 8, dv + (uint64_t)((kk * 2048) >> 4), idesc_pv, kk > 0 ? 1u : acc0);
                                } else {
                                    uint32_t acc = acc0;
#pragma unroll
                                    for (int kk = 0; kk < 4; ++kk) {
                                        if ((l8 >> kk) & 1u) {
                                            mma_ts(d_tmem, a_tmem + kk * 8, dv + (uint64_t)((kk * 2048) >> 4), idesc_pv, acc);
                                            acc = 1u;
                                        }
                                    }
                                }
                            }
                            __syncwarp();
                            ok = mbar_wait_warp(&S.p_ready[w], n_p[w] & 1, abort_flag);
                        }
                        if (ok) {
                            tc_fence_after();
                            if (elect_one()) {
                                if (l8 == 0xFFu) {
#pragma unroll
                                    for (int kk = 4; kk < 8; ++kk)
                                        mma_ts(d_tmem, a_tmem + kk * 8, dv + (uint64_t)((kk * 2048) >> 4), idesc_pv, 1u);
                                } else {
                                    uint32_t acc = (acc0 || (l8 & 0x0Fu)) ? 1u : 0u;
#pragma unroll
                                    for (int kk = 4; kk < 8; ++kk) {
                                        if ((l8 >> kk) & 1u) {
                                            mma_ts(d_tmem, a_tmem + kk * 8, dv + (uint64_t)((kk * 2048) >> 4), idesc_pv, acc);
                                            acc = 1u;
                                        }
                                    }
                                }
                                tc_commit(&S.o_done[w]);
                            }
                            __syncwarp();
                            o_started[w] = o_started[w] || l8 != 0u;
                            ++n_p[w];
                        }
                    }
                    if (ok && use_bit(next, w)) {
                        if (!k_ready) {
                            ok = mbar_wait_warp(&S.k_full[nst], ((it + 1) / kStages) & 1, abort_flag);
                            if constexpr (kCompact) fence_proxy_async();
                            if (ok) tc_fence_after();
                            k_ready = true;
                        }
                        if (ok) issue_s(w, nst);
                    }
                }
                if (ok) {
                    if (elect_one()) {
                        tc_commit(&S.v_empty[st]);
                        if (it + 1 < n_iters_u) tc_commit(&S.k_empty[nst]);
                    }
                    __syncwarp();
                }
            }
        }
    }
    // teardown: every role falls through to here, also after a timed-out wait
    tc_fence_before();
    __syncthreads();
    if (warp == kWarpIssuer) {
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

// Token-compacted mode, per (batch, head, pair of query tiles): the list of keys j that some row i of the
// pair's 256 rows keeps, i.e. j <= i < expiry[j] for some i in [i0, i0 + 255]  <=>  j <= i0 + 255 and expiry[j] > max(i0, j).
// At most w + 256 keys qualify. The list is in two parts, each ascending: first the keys that ALL 256 rows keep
// (j <= i0 and expiry[j] >= i0 + 256), then the keys that enter or expire inside the pair's rows. The forward kernel
// needs no order among the columns, and this one leaves the keys that need the per-element test (a few hundred per pair)
// in the last slices instead of a few in every slice. One CTA of 256 threads per list; every warp owns a contiguous
// eighth of the candidate keys, counts its keys of either part in a first pass and writes them from its start positions
// (the sums of the earlier warps' counts) in a second one: one barrier. Padded with -1 to the next multiple of 128.
__global__ void __launch_bounds__(256) compact_lists_kernel(const int32_t* __restrict__ expiry, int* __restrict__ cidx,
                                                            int* __restrict__ ccnt, int L, int npairs, int cap, int causal,
                                                            int q_off, int32_t* __restrict__ status) {
    __shared__ int wcount[2][8];
    const int list = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bh = list / npairs, pair = list % npairs, i0 = q_off + pair * 256;
    if (!causal && pair != 0) return;                    // non-causal: the head's one list is that of its first pair
    const int32_t* e = expiry + (size_t)bh * L;
    int* out = cidx + (size_t)list * cap;
    const int jend = causal ? min(L, i0 + 256) : L;     // non-causal: key j is kept by the rows i < expiry[j], whatever j
    const int seg = (((jend + 7) / 8 + 31) / 32) * 32, j0 = warp * seg, j1 = min(jend, j0 + seg);
    // 0: not in the list, 1: kept by every row of the pair, 2: kept by some
    auto kind = [&](int j) {
        if (j >= j1) return 0;
        const int ej = e[j], first = causal ? j : 0;
        if (ej <= max(i0, first)) return 0;
        return (first <= i0 && ej >= i0 + 256) ? 1 : 2;
    };
    int c1 = 0, c2 = 0;
    for (int base = j0; base < j1; base += 32) {
        const int k = kind(base + lane);
        c1 += __popc(__ballot_sync(0xffffffffu, k == 1));
        c2 += __popc(__ballot_sync(0xffffffffu, k == 2));
    }
    if (lane == 0) { wcount[0][warp] = c1; wcount[1][warp] = c2; }
    __syncthreads();
    int p1 = 0, p2 = 0, n1 = 0, n2 = 0;
#pragma unroll
    for (int wq = 0; wq < 8; ++wq) {
        const int a = wcount[0][wq], bq = wcount[1][wq];
        p1 += wq < warp ? a : 0;
        p2 += wq < warp ? bq : 0;
        n1 += a;
        n2 += bq;
    }
    p2 += n1;                                            // the second part starts behind the first
    for (int base = j0; base < j1; base += 32) {
        const int j = base + lane, k = kind(j);
        const uint32_t b1 = __ballot_sync(0xffffffffu, k == 1), b2 = __ballot_sync(0xffffffffu, k == 2);
        const uint32_t below = (1u << lane) - 1;
        const int at = k == 1 ? p1 + __popc(b1 & below) : p2 + __popc(b2 & below);
        if (k != 0 && at < cap) out[at] = j;
        p1 += __popc(b1);
        p2 += __popc(b2);
    }
    int n = n1 + n2;
    // more kept keys than the list holds (a mask that keeps more than w keys in some row): reported, not truncated silently
    if (n > cap && tid == 0) atomicExch(status, (int32_t)DMA_ERR_MASK_OVERFLOW);
    n = min(n, cap);
    for (int t = n + tid; t < ((n + 127) / 128) * 128 && t < cap; t += 256) out[t] = -1;
    if (tid == 0) ccnt[list] = n;
}

static int compact_cap(const Prob& P) { return ((P.w + 256 + 127) / 128) * 128; }
static size_t compact_lists(const Prob& P) { return (size_t)P.B * P.Hq * ((P.Tr + 1) / 2); }

size_t tc_fwd_ws_bytes(const Prob& P) {
    if (!(P.flags & DMA_FLAG_COMPACT_KV)) return kWsHeaderBytes;
    const size_t cnt_bytes = ((compact_lists(P) * sizeof(int) + 255) / 256) * 256;
    return kWsHeaderBytes + cnt_bytes + compact_lists(P) * compact_cap(P) * sizeof(int);
}

int launch_tc_fwd(const Prob& P, const void* Q, const void* K, const void* V, const float* bias,
                  const int32_t* expiry, const uint32_t* bitmap, void* O, float* lse, void* ws, cudaStream_t st) {
    const bool compact = (P.flags & DMA_FLAG_COMPACT_KV) != 0;
    if (P.Tc > kMaxSched) return DMA_ERR_UNSUPPORTED;
    const bool block_skip = (P.flags & DMA_FLAG_BLOCK_SKIP) != 0;
    auto kern = P.d == 128 ? (compact ? (block_skip ? fwd_kernel<true, true, 128> : fwd_kernel<true, false, 128>)
                                      : (block_skip ? fwd_kernel<false, true, 128> : fwd_kernel<false, false, 128>))
                           : (compact ? (block_skip ? fwd_kernel<true, true, 64> : fwd_kernel<true, false, 64>)
                                      : (block_skip ? fwd_kernel<false, true, 64> : fwd_kernel<false, false, 64>));
    {
        cudaFuncAttributes fa;       // (before anything is enqueued)
        if (cudaFuncGetAttributes(&fa, kern) != cudaSuccess || fa.numRegs != kLaunchRegs) return DMA_ERR_CUDA;
    }
    CUtensorMap tmQ, tmK, tmV;
    int rc;
    const int Trq = (P.Lq + 127) / 128, npairs = (Trq + 1) / 2;
    if ((P.Lq != P.L || P.q_off != 0) && !compact) return DMA_ERR_UNSUPPORTED;
    if ((rc = make_tmap_bf16(&tmQ, Q, P.B, P.Lq, P.Hq, P.d, P.qs, 128))) return rc;
    FwdParams fp;
    fp.cidx = nullptr; fp.ccnt = nullptr; fp.ccap = 0; fp.Hkv = P.Hkv; fp.causal = P.causal;
    fp.Lq = P.Lq; fp.q_off = P.q_off; fp.Trq = Trq;
    if (!P.causal && !compact) return DMA_ERR_UNSUPPORTED;
    if (compact) {
        if (compact_cap(P) / 128 > kMaxSched) return DMA_ERR_UNSUPPORTED;
        const size_t nl = (size_t)P.B * P.Hq * npairs;
        int* ccnt = reinterpret_cast<int*>((char*)ws + kWsHeaderBytes);
        int* cidx = reinterpret_cast<int*>((char*)ws + kWsHeaderBytes + ((nl * sizeof(int) + 255) / 256) * 256);
        compact_lists_kernel<<<(unsigned)nl, 256, 0, st>>>(expiry, cidx, ccnt, P.L, npairs, compact_cap(P), P.causal, P.q_off, (int32_t*)ws);
        count_launch();
        fp.cidx = cidx; fp.ccnt = ccnt; fp.ccap = compact_cap(P);
    }
    fp.Kg = (const __nv_bfloat16*)K; fp.Vg = (const __nv_bfloat16*)V;
    if ((rc = make_tmap_bf16(&tmK, K, P.B, P.L, P.Hkv, P.d, P.ks, 128))) return rc;
    if ((rc = make_tmap_bf16(&tmV, V, P.B, P.L, P.Hkv, P.d, P.vs, 128))) return rc;
    fp.bias = bias; fp.expiry = expiry; fp.bitmap = bitmap; fp.O = (__nv_bfloat16*)O; fp.lse = lse;
    fp.status = (int32_t*)ws;
    fp.B = P.B; fp.Hq = P.Hq; fp.G = P.G; fp.L = P.L; fp.Tr = P.Tr; fp.Tc = P.Tc; fp.Wd = P.Wd;
    fp.ignore_bitmap = (P.flags & DMA_FLAG_IGNORE_BITMAP) ? 1 : 0;
    fp.scale_log2 = P.scale * 1.4426950408889634f;
    fp.inv_scale = 1.0f / P.scale;
    fp.rescale_gap = kRescaleThreshold / fp.scale_log2;
    fp.os_b = P.os[0]; fp.os_l = P.os[1]; fp.os_h = P.os[2];
    fp.ks_b = P.ks[0]; fp.ks_l = P.ks[1]; fp.ks_h = P.ks[2]; fp.vs_b = P.vs[0]; fp.vs_l = P.vs[1]; fp.vs_h = P.vs[2];
    const size_t smem = sizeof(SharedStorage) + 1024;
    dim3 grid(P.B * P.Hq, npairs);
    timing_mark(0, false, st);
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DMA_ERR_CUDA;
    kern<<<grid, kThreads, smem, st>>>(tmQ, tmK, tmV, fp);
    timing_mark(0, true, st);
    count_launch();
    return check_launch();
}

}  // namespace dma
