// Tensor-core backward (Sec. 4.3, Alg. 2) for bf16, d = 128 or 64, on sm_100a.
//
// One CTA owns one 128-key tile of one KV head and, as in Alg. 2's outer loop, keeps dK, dV (fp32, tensor memory)
// and dM (registers) for it while walking the query heads of the group and their active query tiles in steps of
// 64 query rows. Everything is computed transposed, keys on the 128 TMEM lanes, so that dM is a per-thread row sum
// and P^T, dS^T feed the dV / dK GEMMs straight from tensor memory:
//   S^T  = K Q^T - lse_i / scale     dP^T = V dO^T - D_i      (smem x smem -> TMEM, 64 columns each; the per-row terms
//                                                              come from a ninth k-step: ones (x) three bf16 terms)
//   P^T  = exp2(c S^T + log2e bias_j) where j <= i < expiry[j], else 0;   dS^T = P^T o dP^T
//   dV  += P^T dO           dK  += dS^T Q                      (TMEM x smem  -> TMEM, 128 columns each)
//   dQ^T = K^T dS^T                                            (smem x smem  -> TMEM, 64 columns), staged in shared memory
//                                                              and added to the fp32 dQ accumulator by bulk reduce-adds
// The dQ accumulator is blocked: 16 rows x 32 channels of one head are 2 KB of consecutive floats, so that a staged
// quarter step leaves as ONE contiguous bulk reduce-add (as a tile of a [B, L, Hq, d] tensor map the same 2 KB were 16
// strided 128-byte rows, and issuing that request took the drain warp ~350 cycles: the drain was as long as the step).
// Shared-memory bandwidth is the scarce resource (operand reads of the smem x smem MMAs alone take ~1400 of a step's
// ~2250 cycles), so the compute warps read nothing from shared memory per element.
// Warp roles (16 warps): warps 0-7 compute (thread = key; warps w and w+4 share the 32 TMEM lanes of quadrant w%4 and
// split the 64 query columns of a step), warps 8-11 dQ drain (thread = channel), warp 12 TMA producer + schedule,
// warps 13 and 14 MMA issuers (S^T, dP^T | dV, dK, dQ^T; whole warps with warp-uniform values, one elected lane
// issues), warp 15 stages the ninth k-step operand of each step's query rows.
// TMEM columns: dK [0,128) dV [128,256) S^T [256,320) dP^T [320,384) P^T [384,416) dS^T [416,448) dQ^T [448,512).
// kD = 64 (its own instantiations): K, V, Q and dO tiles are one swizzled half tile each, S^T and dP^T have four k-steps
// and the ninth, dK and dV take 64 columns. What that frees is spent on the two chains that bound a step at d = 128:
//   - P^T and dS^T are double-buffered (tensor-memory columns [64,128) and the unused half of the V buffer for the
//     shared-memory copy of dS^T), so the compute warps store step n+1 while the MMAs of step n still read step n's;
//   - dQ^T = K^T dS^T keeps M = 128 with the K tile loaded a second time into the unused half of its buffer: lanes
//     64-127 repeat lanes 0-63, so all four drain warps work, two per 32 channels, each on half of the step's rows.
#include <cstdlib>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace dma {
namespace {

using namespace ptx;

constexpr int kStages = 3;
constexpr int kMaxSteps = 8192;              // 64-row steps of one CTA: G * ceil(L / 128) * 2 (L = 131072 with four query heads per KV head)
constexpr int kThreads = 512;
constexpr uint32_t kKVBytes = 128 * 128 * 2;   // K or V tile: two 16 KB halves (channels 0-63 | 64-127)
constexpr uint32_t kQBytes = 64 * 128 * 2;     // Q or dO step tile (64 rows): two 8 KB halves
constexpr int cDK = 0, cDV = 128, cS = 256, cDP = 320, cP = 384, cDS = 416, cDQ = 448;
constexpr int cP1 = 64, cDS1 = 96;             // second P^T / dS^T buffer (d = 64 only: beside the 64 columns of dK)

struct SharedStorage {
    alignas(1024) uint8_t k[kKVBytes];
    alignas(1024) uint8_t v[kKVBytes];
    alignas(1024) uint8_t q[kStages][kQBytes];
    alignas(1024) uint8_t g[kStages][kQBytes];       // dO
    alignas(1024) uint8_t ds[128 * 128];             // dS^T as bf16: [128 keys][64 queries], 128-byte swizzled rows
    alignas(1024) float dq_stage[4][2][16][32];      // dQ per drain warp (32 channels), two buffers of 16 query rows: sources of the TMA reduce-adds
    // Ninth k-step of S^T = K Q^T and dP^T = V dO^T (unswizzled K-major core matrices of 8 rows x 16 bytes): it adds
    // -lse_i / scale to S^T and -D_i to dP^T, each as three bf16 terms, so that the compute warps read finished values
    // from tensor memory and need no per-column vector. `ones` = [zero | rows (1,1,1,0..) | zero] blocks of 128 rows:
    // A operand with the ones in elements 0-2 (block 1, then block 2) or in elements 8-10 (block 0, then block 1).
    // `qext[stage]` = B operand, 64 query rows: elements 0-2 = -lse / scale, elements 8-10 = -D.
    alignas(128) uint8_t ones[3][2048];
    alignas(128) uint8_t qext[kStages][2048];
    uint16_t sched[kMaxSteps];                       // head-in-group << 11 | query tile << 1 | half
    uint64_t kv_full, qd_full[kStages], qd_empty[kStages];
    uint64_t sdp_full, sdp_free, pds_ready[2], pds_free[2], dq_full, dq_free;
    uint32_t tmem_base;
    int n_steps;
    int abort_flag;
};

struct BwdParams {
    const float* lse;
    const float* Dv;
    const float* bias;
    const int32_t* expiry;
    const uint32_t* bitmap;
    int sched_group;            // (batch, head) entries per scheduling group, a divisor of gridDim.x
    float* dQacc;               // fp32, zeroed, blocked: [B, Hq, Lblk, d / 32] blocks of 16 rows x 32 channels = 2 KB, each laid out
                                // as the drain warps stage it: channel c owns 64 bytes (its 16 rows), and the 16-byte chunk of
                                // rows 4q .. 4q + 3 sits at chunk q ^ ((c >> 1) & 3) (a thread = a channel then stores four
                                // 16-byte chunks without bank conflicts, instead of 16 scalars)
    int Lblk;                   // 16-row blocks per head: 8 * Tr (rows padded to whole 128-row tiles)
    __nv_bfloat16* dK;
    __nv_bfloat16* dV;
    float* dM;
    int32_t* status;
    int B, Hq, Hkv, G, L, Tr, Tc, Wd, ignore_bitmap;
    float scale, scale_log2, inv_scale;
    // token-compacted mode: per (batch, query head) a permutation of the keys (padded with L to a multiple of 128) that
    // groups keys of similar lifetime; a CTA owns 128 consecutive entries of one query head's permutation
    const int* perm;
    const int32_t* expiry_all;
    int causal;                // 0: key j is visible to every row (token-compacted mode only): its first row is 0 instead of j
    const __nv_bfloat16* Kg;    // K, V base pointers for the row gathers (ks_*, vs_* strides)
    const __nv_bfloat16* Vg;
    float* dKacc;               // fp32 [B, L, Hkv, 128] accumulators (several query heads add into one KV head's rows)
    float* dVacc;
    int64_t acc_slot;           // 0: the group's heads add into one accumulator with atomics; else: elements between the
                                // per-head slots [G][B, L, Hkv, 128], written with plain stores and summed in head order afterwards
    int64_t ks_b, ks_l, ks_h, vs_b, vs_l, vs_h;
};


// x as three bf16 terms (hi, mid, lo: 24 significant bits) in elements 0-2 of a 16-byte core-matrix row
__device__ __forceinline__ uint4 split3(float x) {
    const __nv_bfloat16 hi = __float2bfloat16_rn(x);
    const float r1 = x - __bfloat162float(hi);
    const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
    const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
    return make_uint4((uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(mid) << 16), (uint32_t)__bfloat16_as_ushort(lo), 0u, 0u);
}

// kCompact: token-compacted mode. The CTA's 128 keys are 128 consecutive entries of one QUERY head's lifetime-sorted
// key permutation instead of 128 consecutive keys of a KV head: keys that live equally long are kept by about the
// same query rows, so the walk over query tiles [first key's tile, last expiry's tile] wastes little. K and V rows
// are gathered once with 16-byte asynchronous copies; dK and dV are added to fp32 accumulators (the query heads of a
// group meet there), dM is written directly.
template <bool kCompact, int kD>
__global__ void __launch_bounds__(kThreads, 1)
bwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
           const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmG, const BwdParams P) {
    static_assert(kD == 128 || kD == 64, "head dimensions of the tensor-core kernels");
    constexpr int kHalves = kD / 64;                 // 64-channel (128-byte) swizzled half tiles per operand tile
    constexpr bool kDouble = kD == 64;               // P^T / dS^T in two buffers used in turn (see the file header)
    extern __shared__ uint8_t smem_raw[];
    SharedStorage& S = *reinterpret_cast<SharedStorage*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);      // warp-uniform to the compiler: role branches stay uniform
    // tile mode: blockIdx.x = (batch, KV head); token-compacted mode: (batch, query head), whose group index is fixed
    // CTAs start in the order of lin: heads of one scheduling group (P.sched_group of them) innermost, then key tiles (key
    // tile 0 has the most query tiles: heaviest first), then the groups
    const int lin = blockIdx.y * gridDim.x + blockIdx.x, per_group = P.sched_group * (int)gridDim.y;
    const int bx = (lin / per_group) * P.sched_group + (lin % per_group) % P.sched_group;
    const int b = bx / (kCompact ? P.Hq : P.Hkv);
    const int hq_c = bx % P.Hq;                        // token-compacted mode only
    const int hk = kCompact ? hq_c / P.G : bx % P.Hkv;
    const int kt = (lin % per_group) / P.sched_group;
    const int j0 = kt * 128;
    const int* my_perm = kCompact ? P.perm + ((size_t)bx * P.Tc + kt) * 128 : nullptr;
    volatile int* abort_flag = &S.abort_flag;
    if constexpr (kCompact) {
        // keys that no row keeps are sorted to the end of the permutation: a tile that starts with one holds nothing else
        const int jf = my_perm[0];
        if (jf >= P.L || P.expiry_all[(size_t)bx * P.L + jf] <= (P.causal ? jf : 0)) return;
    }

    if (tid == 0) {
        mbar_init(&S.kv_full, 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&S.qd_full[s], 2);      // TMA bytes + the staged vectors
            mbar_init(&S.qd_empty[s], 1);
        }
        mbar_init(&S.sdp_full, 1);
        mbar_init(&S.sdp_free, 8);        // one arrival per compute warp (256 serialised arrivals would cost hundreds of cycles)
        for (int u = 0; u < 2; ++u) {
            mbar_init(&S.pds_ready[u], 8);
            mbar_init(&S.pds_free[u], 1);
        }
        mbar_init(&S.dq_full, 1);
        mbar_init(&S.dq_free, 4);         // one arrival per drain warp
        S.abort_flag = 0;
        S.n_steps = 0;
        fence_barrier_init();
    }
    if (warp == 13) {
        tmem_alloc(&S.tmem_base, 512);
        tmem_relinquish();
    }
    if (warp == 12) {
        // schedule: for each query head of the group, the active query tiles (ascending), two 64-row steps each
        if (lane == 0) { prefetch_tmap(&tmQ); prefetch_tmap(&tmK); prefetch_tmap(&tmV); prefetch_tmap(&tmG); }
        int n = 0;
        if constexpr (kCompact) {
            // query tiles from the first key's tile to the tile of the last row that keeps one of the keys
            int jmin = 0x7fffffff, emax = 0;
            for (int t = 0; t < 4; ++t) {
                const int j = my_perm[lane + 32 * t];
                const int e = j < P.L ? P.expiry_all[(size_t)bx * P.L + j] : 0;
                const int first = P.causal ? j : 0;
                if (e > first) { jmin = min(jmin, first); emax = max(emax, e); }
            }
            for (int o = 16; o; o >>= 1) {
                jmin = min(jmin, __shfl_xor_sync(0xffffffffu, jmin, o));
                emax = max(emax, __shfl_xor_sync(0xffffffffu, emax, o));
            }
            if (emax > 0) {
                // The walk goes BACKWARDS, from the last row that keeps one of the keys to the first key's row: the CTAs
                // of neighbouring entries of the permutation share their expiry band, i.e. the END of their walks, and start
                // about together, so walking down from there they pass the same query rows (the Q / dO tiles they load, the
                // dQ accumulator rows they add to) at about the same time, while those are in L2; walking up, each from its
                // own first key, they passed a row at times spread over the life of the whole group.
                const int g = hq_c % P.G, q0 = jmin / 128, q1 = (emax - 1) / 128;
                n = 2 * (q1 - q0 + 1);
                if (q1 * 128 + 64 >= P.L) n -= 1;       // the last tile has one 64-row step only
                n = min(n, kMaxSteps);
                for (int qt = q0 + lane; qt <= q1; qt += 32) {
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf) {
                        const int pos = n - 1 - (2 * (qt - q0) + hf);
                        if (pos >= 0) S.sched[pos] = (uint16_t)((g << 11) | (qt << 1) | hf);
                    }
                }
            }
        } else {
        for (int g = 0; g < P.G; ++g) {
            const int bh = b * P.Hq + hk * P.G + g;
            for (int base = kt; base < P.Tr; base += 32) {
                const int qt = base + lane;
                const bool act = qt < P.Tr && (P.ignore_bitmap || bitmap_test(P.bitmap, P.Tr, P.Wd, bh, qt, kt));
                const int halves = act ? ((qt * 128 + 64 < P.L) ? 2 : 1) : 0;
                // exclusive prefix sum of `halves` over the warp
                int incl = halves;
                for (int o = 1; o < 32; o <<= 1) {
                    int t = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += t;
                }
                const int pos = n + incl - halves;
                for (int hf = 0; hf < halves; ++hf)
                    if (pos + hf < kMaxSteps) S.sched[pos + hf] = (uint16_t)((g << 11) | (qt << 1) | hf);
                n += __shfl_sync(0xffffffffu, incl, 31);
            }
        }
        }
        if (lane == 0) S.n_steps = min(n, kMaxSteps);
    }
    if (warp == 15) {
        // constant A operand of the ninth k-step: zero block | rows (1, 1, 1, 0, ...) | zero block
        for (int r = lane; r < 128; r += 32) {
            *reinterpret_cast<uint4*>(S.ones[0] + r * 16) = make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4*>(S.ones[1] + r * 16) = make_uint4(0x3F803F80u, 0x00003F80u, 0u, 0u);
            *reinterpret_cast<uint4*>(S.ones[2] + r * 16) = make_uint4(0u, 0u, 0u, 0u);
        }
        fence_proxy_async();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = S.tmem_base;
    const int n_steps = S.n_steps;

    if (warp < 8) {
        // ============================ compute group: thread = key j, 32 of the step's 64 query columns ============================
        const int quad = warp & 3, hsel = warp >> 2;
        const int r = quad * 32 + lane;                     // key within the tile = TMEM lane
        const int j = kCompact ? my_perm[r] : j0 + r;           // token-compacted mode: padding entries hold L
        const int jf = (kCompact && !P.causal) ? 0 : j;         // first row that can see the key
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        float bj = 0.0f;
        float2 dm2 = make_float2(0.0f, 0.0f);
        int len = 0, cur_g = -1;
        bool ok = true;
        for (int n = 0; n < n_steps && ok; ++n) {
            const uint32_t e = S.sched[n];
            const int g = (int)(e >> 11), i0 = (int)((e >> 1) & 0x3FF) * 128 + (int)(e & 1) * 64;
            const int st = n % kStages;
            if (g != cur_g) {
                const int bh = b * P.Hq + hk * P.G + g;
                if (cur_g >= 0 && j < P.L) atomicAdd(&P.dM[(size_t)(bh - (g - cur_g)) * P.L + j], dm2.x + dm2.y);
                dm2 = make_float2(0.0f, 0.0f);
                bj = j < P.L ? P.bias[(size_t)bh * P.L + j] * 1.4426950408889634f : 0.0f;
                len = j < P.L ? max(0, P.expiry[(size_t)bh * P.L + j] - jf) : 0;
                cur_g = g;
            }
            // (S^T and dP^T were issued after the step's Q / dO stage was full: nothing else of that stage is read here)
            ok = mbar_wait_warp(&S.sdp_full, n & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            uint32_t sr[32], pr[32];
            tmem_ld32(tmem + lane_base + cS + hsel * 32, sr);
            tmem_ld32(tmem + lane_base + cDP + hsel * 32, pr);
            tc_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&S.sdp_free);
            // valid columns of this thread within its 32: col in [lo, lo + width)
            const int c0 = hsel * 32;
            const int lo = max(0, jf - i0 - c0);
            const int width = max(0, min(32, jf - i0 - c0 + len) - lo);
            // Almost every (key, 32-row group) pair is all-or-nothing: then the mask is one additive term per thread
            // (0 or -inf) and the per-element test is skipped. Warps with a partly kept key take the general loop.
            const bool uniform = __all_sync(0xffffffffu, width == 0 || (lo == 0 && width == 32));
            uint32_t pp[16], dd[16];
            const float2 sc2 = make_float2(P.scale_log2, P.scale_log2);
            if (uniform) {
                const float be = width ? bj : -INFINITY;
                const float2 bj2 = make_float2(be, be);
#pragma unroll
                for (int c = 0; c < 32; c += 4) {
                    const float2 x0 = fma2(make_float2(__uint_as_float(sr[c]), __uint_as_float(sr[c + 1])), sc2, bj2);
                    const float2 x1 = fma2(make_float2(__uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3])), sc2, bj2);
                    const float2 t0 = make_float2(__uint_as_float(pr[c]), __uint_as_float(pr[c + 1]));
                    const float2 t1 = make_float2(__uint_as_float(pr[c + 2]), __uint_as_float(pr[c + 3]));
                    const float2 p0 = make_float2(ex2(x0.x), ex2(x0.y)), p1 = make_float2(ex2(x1.x), ex2(x1.y));
                    const float2 d0 = mul2(p0, t0), d1 = mul2(p1, t1);
                    dm2 = add2(dm2, add2(d0, d1));
                    pp[(c >> 1)] = pack_bf16(p0.x, p0.y);
                    pp[(c >> 1) + 1] = pack_bf16(p1.x, p1.y);
                    dd[(c >> 1)] = pack_bf16(d0.x, d0.y);
                    dd[(c >> 1) + 1] = pack_bf16(d1.x, d1.y);
                }
            } else {
                const float2 bj2 = make_float2(bj, bj);
#pragma unroll
                for (int c = 0; c < 32; c += 4) {
                    const float2 x0 = fma2(make_float2(__uint_as_float(sr[c]), __uint_as_float(sr[c + 1])), sc2, bj2);
                    const float2 x1 = fma2(make_float2(__uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3])), sc2, bj2);
                    const float2 t0 = make_float2(__uint_as_float(pr[c]), __uint_as_float(pr[c + 1]));
                    const float2 t1 = make_float2(__uint_as_float(pr[c + 2]), __uint_as_float(pr[c + 3]));
                    float p[4] = {ex2(x0.x), ex2(x0.y), ex2(x1.x), ex2(x1.y)};
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const bool valid = (unsigned)(c + u - lo) < (unsigned)width;
                        p[u] = valid ? p[u] : 0.0f;
                    }
                    const float2 d0 = mul2(make_float2(p[0], p[1]), t0), d1 = mul2(make_float2(p[2], p[3]), t1);
                    dm2 = add2(dm2, add2(d0, d1));
                    pp[(c >> 1)] = pack_bf16(p[0], p[1]);
                    pp[(c >> 1) + 1] = pack_bf16(p[2], p[3]);
                    dd[(c >> 1)] = pack_bf16(d0.x, d0.y);
                    dd[(c >> 1) + 1] = pack_bf16(d1.x, d1.y);
                }
            }
            // the dV / dK / dQ GEMMs that last used this P^T / dS^T buffer (TMEM and smem) must have finished reading it:
            // those of the previous step, or with two buffers those of the step before it
            const int pb = kDouble ? (n & 1) : 0;
            if (kDouble) { if (n > 1) ok = mbar_wait_warp(&S.pds_free[pb], ((n >> 1) - 1) & 1, abort_flag); }
            else if (n > 0) ok = mbar_wait_warp(&S.pds_free[0], (n - 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            tmem_st16(tmem + lane_base + (pb ? cP1 : cP) + hsel * 16, pp);
            tmem_st16(tmem + lane_base + (pb ? cDS1 : cDS) + hsel * 16, dd);
            {   // dS^T row r -> shared memory: 16-byte chunk q of the row sits at q XOR (row % 8) (128-byte swizzle)
                uint8_t* row = (pb ? S.v + kKVBytes / 2 : S.ds) + r * 128;
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    *reinterpret_cast<uint4*>(row + (((hsel * 4 + q) ^ (r & 7)) << 4)) = make_uint4(dd[4 * q], dd[4 * q + 1], dd[4 * q + 2], dd[4 * q + 3]);
            }
            fence_proxy_async();
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&S.pds_ready[pb]);
        }
        if (cur_g >= 0 && j < P.L) atomicAdd(&P.dM[(size_t)(b * P.Hq + hk * P.G + cur_g) * P.L + j], dm2.x + dm2.y);
        // epilogue: dK (scaled) and dV rows to global memory; warps w and w+4 each write one half of the channels
        if (ok && n_steps > 0)
            ok = kDouble ? mbar_wait_warp(&S.pds_free[(n_steps - 1) & 1], ((n_steps - 1) >> 1) & 1, abort_flag)
                         : mbar_wait_warp(&S.pds_free[0], (n_steps - 1) & 1, abort_flag);
        if (ok) {
            tc_fence_after();
            __nv_bfloat16* dk = P.dK + b * P.ks_b + (int64_t)j * P.ks_l + hk * P.ks_h;
            __nv_bfloat16* dv = P.dV + b * P.vs_b + (int64_t)j * P.vs_l + hk * P.vs_h;
            const size_t arow = ((size_t)(b * P.L + min(j, P.L - 1)) * P.Hkv + hk) * kD +      // accumulator row (compact mode)
                                (kCompact ? (size_t)(hq_c % P.G) * (size_t)P.acc_slot : 0);
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                const float mul = which == 0 ? P.scale : 1.0f;
                __nv_bfloat16* out = which == 0 ? dk : dv;
                float* acc = (which == 0 ? P.dKacc : P.dVacc) + arow;
#pragma unroll
                for (int cc = 0; cc < kHalves; ++cc) {
                    const int c = hsel * kHalves + cc;
                    uint32_t o[32];
                    if (n_steps > 0) {
                        tmem_ld32(tmem + lane_base + (which == 0 ? cDK : cDV) + c * 32, o);
                        tc_wait_ld();
                    } else {
#pragma unroll
                        for (int u = 0; u < 32; ++u) o[u] = 0;
                    }
                    if constexpr (kCompact) {
                        // unscaled sums into the fp32 accumulators: the group's query heads add into the same rows
                        if (j < P.L && n_steps > 0) {
                            if (P.acc_slot) {          // this (key, query head) pair is written by this thread alone
#pragma unroll
                                for (int u = 0; u < 32; u += 4)
                                    *reinterpret_cast<float4*>(acc + c * 32 + u) = make_float4(__uint_as_float(o[u]), __uint_as_float(o[u + 1]),
                                                                                              __uint_as_float(o[u + 2]), __uint_as_float(o[u + 3]));
                            } else {
#pragma unroll
                                for (int u = 0; u < 32; u += 4)
                                    red_add_v4(acc + c * 32 + u, __uint_as_float(o[u]), __uint_as_float(o[u + 1]), __uint_as_float(o[u + 2]),
                                               __uint_as_float(o[u + 3]));
                            }
                        }
                    } else if (j < P.L) {
#pragma unroll
                        for (int u = 0; u < 32; u += 8) {
                            uint4 pkt;
                            pkt.x = pack_bf16(__uint_as_float(o[u]) * mul, __uint_as_float(o[u + 1]) * mul);
                            pkt.y = pack_bf16(__uint_as_float(o[u + 2]) * mul, __uint_as_float(o[u + 3]) * mul);
                            pkt.z = pack_bf16(__uint_as_float(o[u + 4]) * mul, __uint_as_float(o[u + 5]) * mul);
                            pkt.w = pack_bf16(__uint_as_float(o[u + 6]) * mul, __uint_as_float(o[u + 7]) * mul);
                            *reinterpret_cast<uint4*>(out + c * 32 + u) = pkt;
                        }
                    }
                }
            }
        }
    } else if (warp < 12) {
        // ============================ dQ drain group: thread = channel c, columns = query rows ============================
        // Each warp owns 32 channels and its own pair of staging buffers (16 query rows each, used in turn), so the
        // warps never wait for each other: a buffer is rewritten once the reduce-add issued from it two groups ago has
        // finished reading it.
        // d = 64: lanes 64-127 of dQ^T repeat lanes 0-63 (the K tile sits in both halves of its buffer), so warps 2 and 3
        // own the same channels as warps 0 and 1 and take the second half of the step's rows.
        const int dw = warp & 3;
        constexpr int kQuarters = kD == 64 ? 2 : 4;                     // quarter steps per warp
        const int ch = kD == 64 ? (dw & 1) : dw, qr0 = kD == 64 ? (dw >> 1) * 2 : 0;
        const uint32_t lane_base = (uint32_t)(dw * 32) << 16;
        bool ok = true;
        for (int n = 0; n < n_steps && ok; ++n) {
            const uint32_t e = S.sched[n];
            const int g = (int)(e >> 11), i0 = (int)((e >> 1) & 0x3FF) * 128 + (int)(e & 1) * 64;
            ok = mbar_wait_warp(&S.dq_full, n & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            uint32_t v[kQuarters * 16];
#pragma unroll
            for (int c = 0; c < kQuarters / 2; ++c)
                tmem_ld32(tmem + lane_base + cDQ + qr0 * 16 + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&v[c * 32]));
            tc_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&S.dq_free);
#pragma unroll
            for (int q = 0; q < kQuarters; ++q) {      // quarter steps of 16 query rows, two staging buffers in turn
                const int qr = qr0 + q;
                if (lane == 0) bulk_wait_read_1(); __syncwarp();
                {   // this thread's channel, 16 rows: four 16-byte stores (see BwdParams::dQacc for the block's layout)
                    uint8_t* line = reinterpret_cast<uint8_t*>(&S.dq_stage[dw][q & 1][0][0]) + lane * 64;
#pragma unroll
                    for (int qq = 0; qq < 4; ++qq)
                        *reinterpret_cast<uint4*>(line + ((qq ^ ((lane >> 1) & 3)) << 4)) =
                            make_uint4(v[q * 16 + 4 * qq], v[q * 16 + 4 * qq + 1], v[q * 16 + 4 * qq + 2], v[q * 16 + 4 * qq + 3]);
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0 && i0 + qr * 16 < P.L) {       // (rows beyond L inside the block land in the accumulator's padding)
                    float* blk = P.dQacc + ((((size_t)(b * P.Hq + hk * P.G + g) * P.Lblk + (i0 >> 4) + qr) * (kD / 32) + ch) << 9);
                    bulk_reduce_add_f32(blk, &S.dq_stage[dw][q & 1][0][0], 2048);
                }
                if (lane == 0) bulk_commit();
            }
        }
        if (lane == 0) bulk_wait_all();
    } else {
        if (warp == 12) {
            // ============================ producer ============================
            if constexpr (kCompact) {
                if (n_steps > 0) {
                // gather the CTA's 128 K and V rows into the swizzled tile layout (8 lanes per 128-byte half row,
                // 4 rows per instruction; padding entries are zero-filled)
                const int rsub = lane >> 3, c = lane & 7;
#pragma unroll 4
                for (int q = 0; q < 32; ++q) {
                    const int r = 4 * q + rsub, j = my_perm[r];
                    const int64_t jr = min(j, P.L - 1);
                    const int64_t krow = b * P.ks_b + jr * P.ks_l + hk * P.ks_h + c * 8, vrow = b * P.vs_b + jr * P.vs_l + hk * P.vs_h + c * 8;
                    const uint32_t off = r * 128 + ((c ^ (r & 7)) << 4);
                    const int nb = j < P.L ? 16 : 0;
                    cp_async16(S.k + off, P.Kg + krow, nb);
                    cp_async16(S.k + off + kKVBytes / 2, P.Kg + krow + (kD == 128 ? 64 : 0), nb);     // d = 64: the same 64 channels once more
                    cp_async16(S.v + off, P.Vg + vrow, nb);
                    if constexpr (kD == 128) cp_async16(S.v + off + kKVBytes / 2, P.Vg + vrow + 64, nb);
                }
                cp_async_wait_all();
                fence_proxy_async();
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&S.kv_full);
            } else if (lane == 0) {
                mbar_arrive_expect_tx(&S.kv_full, (kD == 128 ? 4 : 3) * (kKVBytes / 2));
                for (int hf = 0; hf < 2; ++hf) {           // d = 64: both halves of the K buffer hold the same 64 channels
                    tma_load_4d(&S.k[hf * (kKVBytes / 2)], &tmK, &S.kv_full, kD == 128 ? hf * 64 : 0, j0, hk, b);
                    if (hf < kHalves) tma_load_4d(&S.v[hf * (kKVBytes / 2)], &tmV, &S.kv_full, hf * 64, j0, hk, b);
                }
            }
            bool ok = true;
            for (int n = 0; n < n_steps && ok; ++n) {
                const uint32_t e = S.sched[n];
                const int h = hk * P.G + (int)(e >> 11), i0 = (int)((e >> 1) & 0x3FF) * 128 + (int)(e & 1) * 64;
                const int st = n % kStages;
                if (n >= kStages) ok = mbar_wait_warp(&S.qd_empty[st], ((n / kStages) - 1) & 1, abort_flag);
                if (!ok) break;
                if (lane == 0) {
                    mbar_arrive_expect_tx(&S.qd_full[st], kHalves * kQBytes);
                    for (int hf = 0; hf < kHalves; ++hf) {
                        tma_load_4d(&S.q[st][hf * (kQBytes / 2)], &tmQ, &S.qd_full[st], hf * 64, i0, h, b);
                        tma_load_4d(&S.g[st][hf * (kQBytes / 2)], &tmG, &S.qd_full[st], hf * 64, i0, h, b);
                    }
                }
            }
            for (int n = max(0, n_steps - kStages); n < n_steps && ok; ++n)
                ok = mbar_wait_warp(&S.qd_empty[n % kStages], (n / kStages) & 1, abort_flag);
        } else if (warp == 15) {
            // ============================ stager: ninth k-step B operand (-lse / scale, -D) of each step's query rows, loaded one step ahead ============================
            auto fetch = [&](int n, float (&lv)[2], float (&dv)[2]) {
                const uint32_t e = S.sched[n];
                const int h = hk * P.G + (int)(e >> 11), i0 = (int)((e >> 1) & 0x3FF) * 128 + (int)(e & 1) * 64;
                const size_t rowbase = (size_t)(b * P.Hq + h) * P.L;
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const int i = i0 + lane + 32 * t;
                    lv[t] = i < P.L ? P.lse[rowbase + i] : 0.0f;
                    dv[t] = i < P.L ? P.Dv[rowbase + i] : 0.0f;
                }
            };
            float lv[2] = {0.f, 0.f}, dv[2] = {0.f, 0.f};
            if (n_steps > 0) fetch(0, lv, dv);
            bool ok = true;
            for (int n = 0; n < n_steps && ok; ++n) {
                const int st = n % kStages;
                float ln[2] = {0.f, 0.f}, dn[2] = {0.f, 0.f};
                if (n + 1 < n_steps) fetch(n + 1, ln, dn);
                if (n >= kStages) ok = mbar_wait_warp(&S.qd_empty[st], ((n / kStages) - 1) & 1, abort_flag);
                if (!ok) break;
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const int r = lane + 32 * t;
                    uint8_t* row = S.qext[st] + (r >> 3) * 256 + (r & 7) * 16;
                    *reinterpret_cast<uint4*>(row) = split3(-lv[t] * P.inv_scale);        // elements 0-2: -lse_i / scale
                    *reinterpret_cast<uint4*>(row + 128) = split3(-dv[t]);                // elements 8-10: -D_i
                    lv[t] = ln[t];
                    dv[t] = dn[t];
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(&S.qd_full[st]);
            }
        } else if (warp == 13) {
            // ============================ MMA issuer 1: S^T = K Q^T, dP^T = V dO^T ============================
            // (two issuing warps: every hand-over between them and the other groups is an explicit mbarrier, nothing
            //  relies on the order of their MMAs. Each walks the schedule as a whole warp with warp-uniform values, so
            //  that descriptors and counters stay in the uniform datapath; one elected lane issues.)
            constexpr uint32_t id_sdp = idesc_bf16(128, 64, 0, 0);     // K|V (K-major) x Q|dO (K-major)       -> 128 x 64
            const uint64_t dK = smem_desc_sw128(smem_u32(S.k), 16, 1024), dV = smem_desc_sw128(smem_u32(S.v), 16, 1024);
            const uint64_t dQ0 = smem_desc_sw128(smem_u32(S.q[0]), 16, 1024), dG0 = smem_desc_sw128(smem_u32(S.g[0]), 16, 1024);
            // ninth k-step: 8-row groups 128 bytes apart, second K core matrix one 2 KB block further (A) / 128 bytes further (B)
            const uint64_t dOnesLo = smem_desc_plain(smem_u32(S.ones[1]), 2048, 128), dOnesHi = smem_desc_plain(smem_u32(S.ones[0]), 2048, 128);
            const uint64_t dX0 = smem_desc_plain(smem_u32(S.qext[0]), 128, 256);
            const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem, 0);
            const int n_steps_u = __shfl_sync(0xffffffffu, n_steps, 0);
            bool ok = mbar_wait_warp(&S.kv_full, 0, abort_flag);
            for (int n = 0; n < n_steps_u && ok; ++n) {
                const int st = n % kStages;
                ok = mbar_wait_warp(&S.qd_full[st], (n / kStages) & 1, abort_flag);
                if (ok && n > 0) ok = mbar_wait_warp(&S.sdp_free, (n - 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint64_t dQ = dQ0 + (uint64_t)(st * (kQBytes >> 4)), dG = dG0 + (uint64_t)(st * (kQBytes >> 4));
                const uint64_t dX = dX0 + (uint64_t)(st * (2048 >> 4));
                if (elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < kD / 16; ++kk)
                        mma_ss(tmem_u + cS, dK + (uint64_t)(((kk >> 2) * (kKVBytes / 2) + (kk & 3) * 32) >> 4),
                               dQ + (uint64_t)(((kk >> 2) * (kQBytes / 2) + (kk & 3) * 32) >> 4), id_sdp, kk > 0);
                    mma_ss(tmem_u + cS, dOnesLo, dX, id_sdp, 1u);          // S^T  += 1 (x) (-lse / scale)
#pragma unroll
                    for (int kk = 0; kk < kD / 16; ++kk)
                        mma_ss(tmem_u + cDP, dV + (uint64_t)(((kk >> 2) * (kKVBytes / 2) + (kk & 3) * 32) >> 4),
                               dG + (uint64_t)(((kk >> 2) * (kQBytes / 2) + (kk & 3) * 32) >> 4), id_sdp, kk > 0);
                    mma_ss(tmem_u + cDP, dOnesHi, dX, id_sdp, 1u);         // dP^T += 1 (x) (-D)
                    tc_commit(&S.sdp_full);
                }
                __syncwarp();
            }
        } else if (warp == 14) {
            // ============================ MMA issuer 2: dV += P^T dO, dK += dS^T Q, dQ^T = K^T dS^T ============================
            constexpr uint32_t id_dkv = idesc_bf16(128, kD, 0, 1);     // P^T|dS^T (TMEM) x dO|Q (MN-major)    -> 128 x d
            constexpr uint32_t id_dq = idesc_bf16(128, 64, 1, 1);      // K^T (MN-major) x dS^T (MN-major)     -> 128 x 64
            const uint64_t dKt = smem_desc_sw128(smem_u32(S.k), kKVBytes / 2, 1024), dDs0 = smem_desc_sw128(smem_u32(S.ds), 16, 1024);
            const uint64_t dDs1 = smem_desc_sw128(smem_u32(S.v + kKVBytes / 2), 16, 1024);      // second dS^T buffer (d = 64)
            const uint64_t dGm0 = smem_desc_sw128(smem_u32(S.g[0]), kQBytes / 2, 1024), dQm0 = smem_desc_sw128(smem_u32(S.q[0]), kQBytes / 2, 1024);
            const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem, 0);
            const int n_steps_u = __shfl_sync(0xffffffffu, n_steps, 0);
            bool ok = true;
            for (int n = 0; n < n_steps_u && ok; ++n) {
                const int st = n % kStages;
                const int pb = kDouble ? (n & 1) : 0;
                ok = mbar_wait_warp(&S.pds_ready[pb], (kDouble ? (n >> 1) : n) & 1, abort_flag);
                if (ok && n > 0) ok = mbar_wait_warp(&S.dq_free, (n - 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t tP = tmem_u + (pb ? cP1 : cP), tDS = tmem_u + (pb ? cDS1 : cDS);
                const uint64_t dDs = pb ? dDs1 : dDs0;
                const uint64_t dGm = dGm0 + (uint64_t)(st * (kQBytes >> 4)), dQm = dQm0 + (uint64_t)(st * (kQBytes >> 4));
                const uint32_t acc0 = n > 0 ? 1u : 0u;
                if (elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)         // 64 query rows = 4 k-steps of 16
                        mma_ts(tmem_u + cDV, tP + kk * 8, dGm + (uint64_t)((kk * 2048) >> 4), id_dkv, kk > 0 ? 1u : acc0);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        mma_ts(tmem_u + cDK, tDS + kk * 8, dQm + (uint64_t)((kk * 2048) >> 4), id_dkv, kk > 0 ? 1u : acc0);
                    tc_commit(&S.qd_empty[st]);            // the dQ GEMM reads K and dS^T only: Q / dO of this stage are free here
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)         // 128 keys = 8 k-steps of 16
                        mma_ss(tmem_u + cDQ, dKt + (uint64_t)((kk * 2048) >> 4), dDs + (uint64_t)((kk * 2048) >> 4), id_dq, kk > 0);
                    tc_commit(&S.pds_free[pb]);
                    tc_commit(&S.dq_full);
                }
                __syncwarp();
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 13) {
        tc_fence_after();
        tmem_dealloc(tmem, 512);
    }
    if (tid == 0 && S.abort_flag) atomicExch(P.status, (int32_t)DMA_ERR_DEVICE_TIMEOUT);
}

// D_i = dO_i . O_i  (Alg. 2): kLanes = d / 8 lanes per (b, h, i), 16-byte loads (a row of 128 bf16 is 16 x 16 bytes)
template <int kLanes>
__global__ void rowdot_bf16_kernel(const __nv_bfloat16* __restrict__ O, const __nv_bfloat16* __restrict__ dO,
                                   float* __restrict__ Dv, int B, int L, int Hq, int64_t os_b, int64_t os_l, int64_t os_h) {
    const long row = (long)blockIdx.x * (blockDim.x / kLanes) + threadIdx.x / kLanes;
    const int sub = threadIdx.x % kLanes;
    float s = 0.0f;
    if (row < (long)B * Hq * L) {
        const int i = row % L, h = (row / L) % Hq, b = row / ((long)L * Hq);
        const int64_t off = b * os_b + (int64_t)i * os_l + h * os_h + sub * 8;
        const uint4 a = *reinterpret_cast<const uint4*>(O + off), g = *reinterpret_cast<const uint4*>(dO + off);
        const uint32_t au[4] = {a.x, a.y, a.z, a.w}, gu[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            s = fmaf(__uint_as_float(au[t] << 16), __uint_as_float(gu[t] << 16), s);
            s = fmaf(__uint_as_float(au[t] & 0xffff0000u), __uint_as_float(gu[t] & 0xffff0000u), s);
        }
    }
    for (int m = kLanes / 2; m; m >>= 1) s += __shfl_xor_sync(0xffffffffu, s, m);
    if (sub == 0 && row < (long)B * Hq * L) Dv[row] = s;
}

// fp32 accumulator [B, L, Hq, d] (unscaled dS K sums) -> softmax scale applied -> bf16 dQ in the caller's layout; 8 elements per thread.
// nslots > 1: the accumulator is nslots copies, slot_stride elements apart, added here in slot order (a fixed order: the
// result is then the same bits from run to run).
__global__ void dq_convert_bf16_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ dQ, size_t n8, int L, int Hq,
                                       int64_t qs_b, int64_t qs_l, int64_t qs_h, float scale, int d, int nslots = 1, int64_t slot_stride = 0) {
    const size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n8) return;
    const size_t e = t * 8;
    const int c = e % d, h = (e / d) % Hq, i = (e / ((size_t)d * Hq)) % L, b = e / ((size_t)d * Hq * L);
    float4 a = *reinterpret_cast<const float4*>(acc + e), bb = *reinterpret_cast<const float4*>(acc + e + 4);
    for (int sl = 1; sl < nslots; ++sl) {
        const float4 a2 = *reinterpret_cast<const float4*>(acc + (size_t)sl * slot_stride + e), b2 = *reinterpret_cast<const float4*>(acc + (size_t)sl * slot_stride + e + 4);
        a.x += a2.x; a.y += a2.y; a.z += a2.z; a.w += a2.w; bb.x += b2.x; bb.y += b2.y; bb.z += b2.z; bb.w += b2.w;
    }
    uint4 o;
    o.x = ptx::pack_bf16(a.x * scale, a.y * scale); o.y = ptx::pack_bf16(a.z * scale, a.w * scale);
    o.z = ptx::pack_bf16(bb.x * scale, bb.y * scale); o.w = ptx::pack_bf16(bb.z * scale, bb.w * scale);
    *reinterpret_cast<uint4*>(dQ + b * qs_b + (int64_t)i * qs_l + h * qs_h + c) = o;
}

// blocked fp32 dQ accumulator (see BwdParams::dQacc) -> softmax scale applied -> bf16 dQ in the caller's layout. One CTA per
// (batch, head, 16-row block); a thread takes two neighbouring channels (they share their chunk position) and four rows:
// two 16-byte loads, four 4-byte stores that the lanes of a warp, consecutive channel pairs, make whole 128-byte lines of.
__global__ void __launch_bounds__(256) dq_unblock_bf16_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ dQ, int L, int Hq,
                                                              int Lblk, int64_t qs_b, int64_t qs_l, int64_t qs_h, float scale, int d) {
    const int t = threadIdx.x, rb = blockIdx.x % Lblk, bh = blockIdx.x / Lblk, h = bh % Hq, b = bh / Hq;
    const int pairs = d >> 1, p = t % pairs, q = t / pairs;            // channel pair, quad of rows
    if (q >= 4) return;
    const int c = 2 * p, cc = c & 31;
    const float* src = acc + ((size_t)bh * Lblk + rb) * (size_t)d * 16 + (c >> 5) * 512 + cc * 16 + ((q ^ ((cc >> 1) & 3)) << 2);
    const float4 x = *reinterpret_cast<const float4*>(src), y = *reinterpret_cast<const float4*>(src + 16);
    const float xs[4] = {x.x, x.y, x.z, x.w}, ys[4] = {y.x, y.y, y.z, y.w};
    __nv_bfloat16* out = dQ + b * qs_b + h * qs_h + c;
#pragma unroll
    for (int rr = 0; rr < 4; ++rr) {
        const int i = rb * 16 + 4 * q + rr;
        if (i < L) *reinterpret_cast<uint32_t*>(out + (int64_t)i * qs_l) = ptx::pack_bf16(xs[rr] * scale, ys[rr] * scale);
    }
}

}  // namespace

// Token-compacted mode: per (batch, query head) a stable counting sort of the keys by the band their expiry falls in
// (band size >= 2048 rows, at most 62 bands; latest expiry first; keys that no row keeps go last). Within a band the
// keys stay in index order, so 128 consecutive entries start at nearby rows and expire within one band of each other:
// on i.i.d. importance at L = 16384, w = 2048 the walk covers 1.4 x the (row, key) pairs actually kept, against 4.3 x
// for tiles of consecutive keys. Padded with L up to Tc * 128.
// One CTA of 1024 threads per (batch, head). Per 1024-key chunk every warp ranks its 32 keys within their class
// (match_any), the per-warp class counts are turned into start positions by 64 threads (one per class, a running sum over
// the 32 warps and over the chunks), and every key is written to its place: stable in key order, three barriers per chunk.
__global__ void __launch_bounds__(1024) lifetime_perm_kernel(const int32_t* __restrict__ expiry, int* __restrict__ perm, int L, int Tc, int causal) {
    __shared__ int hist[64];
    __shared__ int offs[64];                 // next free position of each class
    __shared__ int cnt[32][64];              // per warp and class: keys in this chunk, then their start position
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t* e = expiry + (size_t)blockIdx.x * L;
    int* out = perm + (size_t)blockIdx.x * Tc * 128;
    const int band = max(2048, (L + 61) / 62);
    auto cls = [&](int j) { return e[j] > (causal ? j : 0) ? 1 + (e[j] - 1) / band : 0; };
    if (tid < 64) hist[tid] = 0;
    __syncthreads();
    for (int j = tid; j < L; j += 1024) atomicAdd(&hist[cls(j)], 1);
    __syncthreads();
    if (tid == 0) {
        int run = 0;
        for (int c = 63; c >= 0; --c) { offs[c] = run; run += hist[c]; }
    }
    __syncthreads();
    for (int base = 0; base < L; base += 1024) {
        const int j = base + tid;
        const int c = j < L ? cls(j) : -1;
        const uint32_t same = __match_any_sync(0xffffffffu, c);
        const int leader = __ffs(same) - 1, rank = __popc(same & ((1u << lane) - 1));
        cnt[warp][lane] = 0;
        cnt[warp][lane + 32] = 0;
        __syncwarp();
        if (lane == leader && c >= 0) cnt[warp][c] = __popc(same);
        __syncthreads();
        if (tid < 64) {
            int run = offs[tid];
            for (int w = 0; w < 32; ++w) {
                const int n = cnt[w][tid];
                cnt[w][tid] = run;
                run += n;
            }
            offs[tid] = run;
        }
        __syncthreads();
        if (c >= 0) out[cnt[warp][c] + rank] = j;
        __syncthreads();
    }
    for (int t = L + tid; t < Tc * 128; t += 1024) out[t] = L;
}

// workspace layout: header | D [rows] | dQ accumulator [B x Hq x (Tr x 128) x d] | (token-compacted mode) permutation | dK, dV accumulators
static size_t bwd_rows64(const Prob& P) { return ((((size_t)P.B * P.Hq * P.L) + 63) / 64) * 64; }
static size_t bwd_acc_floats(const Prob& P) { return (size_t)P.B * P.Hq * P.Tr * 128 * P.d; }     // rows padded to whole query tiles
static size_t bwd_perm_ints(const Prob& P) { return (((size_t)P.B * P.Hq * P.Tc * 128) + 63) / 64 * 64; }

size_t tc_bwd_ws_bytes(const Prob& P) {
    size_t n = kWsHeaderBytes + (bwd_rows64(P) + bwd_acc_floats(P)) * sizeof(float);
    const size_t slots = (P.flags & DMA_FLAG_DETERMINISTIC) ? (size_t)P.G : 1;      // per-head dK / dV accumulators
    if (P.flags & DMA_FLAG_COMPACT_KV) n += bwd_perm_ints(P) * sizeof(int) + 2 * slots * (size_t)P.B * P.L * P.Hkv * P.d * sizeof(float);
    return n;
}

int launch_tc_bwd(const Prob& P, const void* Q, const void* K, const void* V, const void* O, const void* dO,
                  const float* lse, const float* bias, const int32_t* expiry, const uint32_t* bitmap, void* dQ,
                  void* dK, void* dV, float* dM, void* ws, cudaStream_t st) {
    const bool compact = (P.flags & DMA_FLAG_COMPACT_KV) != 0;
    if (!P.causal && !compact) return DMA_ERR_UNSUPPORTED;
    if ((size_t)P.G * P.Tr * 2 > (size_t)kMaxSteps || P.G > 16 || P.Tr > 1024) return DMA_ERR_UNSUPPORTED;
    const size_t rows = (size_t)P.B * P.Hq * P.L, nq = rows * P.d, nkv = (size_t)P.B * P.L * P.Hkv * P.d;
    float* Dv = reinterpret_cast<float*>((char*)ws + kWsHeaderBytes);
    float* acc = Dv + bwd_rows64(P);
    int* perm = reinterpret_cast<int*>(acc + bwd_acc_floats(P));
    const size_t slots = (compact && (P.flags & DMA_FLAG_DETERMINISTIC)) ? (size_t)P.G : 1;
    float* accK = reinterpret_cast<float*>(perm + bwd_perm_ints(P));
    float* accV = accK + slots * nkv;
    CUtensorMap tmQ, tmK, tmV, tmG;
    int rc;
    if ((rc = make_tmap_bf16(&tmQ, Q, P.B, P.L, P.Hq, P.d, P.qs, 64))) return rc;
    if ((rc = make_tmap_bf16(&tmG, dO, P.B, P.L, P.Hq, P.d, P.os, 64))) return rc;
    if ((rc = make_tmap_bf16(&tmK, K, P.B, P.L, P.Hkv, P.d, P.ks, 128))) return rc;
    if ((rc = make_tmap_bf16(&tmV, V, P.B, P.L, P.Hkv, P.d, P.vs, 128))) return rc;
    if (P.d == 128)
        rowdot_bf16_kernel<16><<<(unsigned)((rows + 15) / 16), 256, 0, st>>>((const __nv_bfloat16*)O, (const __nv_bfloat16*)dO, Dv, P.B, P.L, P.Hq,
                                                                            P.os[0], P.os[1], P.os[2]);
    else
        rowdot_bf16_kernel<8><<<(unsigned)((rows + 31) / 32), 256, 0, st>>>((const __nv_bfloat16*)O, (const __nv_bfloat16*)dO, Dv, P.B, P.L, P.Hq,
                                                                           P.os[0], P.os[1], P.os[2]);
    if (cudaMemsetAsync(acc, 0, bwd_acc_floats(P) * sizeof(float), st) != cudaSuccess) return DMA_ERR_CUDA;
    if (cudaMemsetAsync(dM, 0, rows * sizeof(float), st) != cudaSuccess) return DMA_ERR_CUDA;   // two partial sums are added per key
    if (compact) {
        if (cudaMemsetAsync(accK, 0, 2 * slots * nkv * sizeof(float), st) != cudaSuccess) return DMA_ERR_CUDA;
        lifetime_perm_kernel<<<P.B * P.Hq, 1024, 0, st>>>(expiry, perm, P.L, P.Tc, P.causal);
        count_launch();
    }
    BwdParams bp;
    bp.lse = lse; bp.Dv = Dv; bp.bias = bias; bp.expiry = expiry; bp.bitmap = bitmap; bp.dQacc = acc; bp.Lblk = P.Tr * 8;
    bp.dK = (__nv_bfloat16*)dK; bp.dV = (__nv_bfloat16*)dV; bp.dM = dM; bp.status = (int32_t*)ws;
    bp.B = P.B; bp.Hq = P.Hq; bp.Hkv = P.Hkv; bp.G = P.G; bp.L = P.L; bp.Tr = P.Tr; bp.Tc = P.Tc; bp.Wd = P.Wd;
    bp.ignore_bitmap = (P.flags & DMA_FLAG_IGNORE_BITMAP) ? 1 : 0;
    {
        // CTA start order: all key tiles of a few (batch, KV head) entries before the next few, so that the
        // rows those CTAs stream (Q, dO) and add to (the fp32 dQ accumulator: 8 bytes per element and query head in all)
        // stay in L2 while they are in use. About 160 MB of such rows per group was the best of the orders measured at
        // L = 16384 with 32 / 8 heads (two KV heads per group: 1.3 % faster in a long run than all eight at once; one
        // KV head per group starts the heaviest CTAs of the last group too late).
        const int gx = compact ? P.B * P.Hq : P.B * P.Hkv;
        int sg = gx;
        {
            const double per_entry = (double)(compact ? 1 : P.G) * P.L * P.d * 8;     // token-compacted mode: an entry is one query head
            // (token-compacted mode, eight heads at L = 16384: 1.69 ms against 1.74 with four and 1.82 with sixteen, once the
            //  CTAs walk backwards; with the forward walk four at a time was the best, 1.77 against 1.88)
            int want = (int)(160.0 * 1024 * 1024 / per_entry);
            want = want < 1 ? 1 : want;
            for (sg = want < gx ? want : gx; gx % sg; --sg) {}
        }
        bp.sched_group = sg;
    }
    bp.scale = P.scale; bp.scale_log2 = P.scale * 1.4426950408889634f; bp.inv_scale = 1.0f / P.scale;
    bp.ks_b = P.ks[0]; bp.ks_l = P.ks[1]; bp.ks_h = P.ks[2]; bp.vs_b = P.vs[0]; bp.vs_l = P.vs[1]; bp.vs_h = P.vs[2];
    bp.perm = perm; bp.expiry_all = expiry; bp.causal = P.causal; bp.Kg = (const __nv_bfloat16*)K; bp.Vg = (const __nv_bfloat16*)V;
    bp.dKacc = accK; bp.dVacc = accV; bp.acc_slot = slots > 1 ? (int64_t)nkv : 0;
    const size_t smem = sizeof(SharedStorage) + 1024;
    timing_mark(1, false, st);
    if (compact) {
        auto kern = P.d == 128 ? bwd_kernel<true, 128> : bwd_kernel<true, 64>;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DMA_ERR_CUDA;
        kern<<<dim3(P.B * P.Hq, P.Tc), kThreads, smem, st>>>(tmQ, tmK, tmV, tmG, bp);
        timing_mark(1, true, st);
        const int nb = (int)((nkv / 8 + 255) / 256);
        dq_convert_bf16_kernel<<<nb, 256, 0, st>>>(accK, (__nv_bfloat16*)dK, nkv / 8, P.L, P.Hkv, P.ks[0], P.ks[1], P.ks[2], P.scale, P.d, (int)slots, (int64_t)nkv);
        dq_convert_bf16_kernel<<<nb, 256, 0, st>>>(accV, (__nv_bfloat16*)dV, nkv / 8, P.L, P.Hkv, P.vs[0], P.vs[1], P.vs[2], 1.0f, P.d, (int)slots, (int64_t)nkv);
        count_launch(2);
    } else {
        auto kern = P.d == 128 ? bwd_kernel<false, 128> : bwd_kernel<false, 64>;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DMA_ERR_CUDA;
        kern<<<dim3(P.B * P.Hkv, P.Tc), kThreads, smem, st>>>(tmQ, tmK, tmV, tmG, bp);
        timing_mark(1, true, st);
    }
    dq_unblock_bf16_kernel<<<(unsigned)((size_t)P.B * P.Hq * P.Tr * 8), 256, 0, st>>>(acc, (__nv_bfloat16*)dQ, P.L, P.Hq, P.Tr * 8, P.qs[0], P.qs[1], P.qs[2], P.scale, P.d);
    count_launch(3);
    return check_launch();
}

}  // namespace dma
