// Mask generation (Sec. 4.1): value projection + gating (Eq. delta_calc), exact per-row top-w selection in
// compact "expiry" form (Eq. mask_combine read per query row over the causally visible keys), and the
// (query tile, key tile) activity bitmap (the Judge test of Alg. 1 / Alg. 2).
//
// Kernels
//   delta_kernel        V read once (HBM-bound); z, softplus, exp in a fixed fp32 operation order
//   chunk_sort_kernel   256-key chunks of (delta bits, ~index) keys sorted in shared memory
//   tree_block_kernel, tree_merge_kernel, expiry_tree_kernel
//                       selection as a rank tree: the merge passes that finish the sort leave one bit per key and level,
//                       and a key's expiry (the w-th smallest index among the keys that beat it) is a walk of log2(L) steps
//   bitmap_kernel       per key tile: union of the query-tile intervals its keys are kept in
#include <mutex>
#include <utility>
#include <type_traits>

#include "common.cuh"

namespace dma {
namespace {

constexpr int kChunk = 256;   // keys per sorted chunk (= threads of the sort kernel)

// ---- fixed-order fp32 routines: every step is one correctly rounded IEEE operation -----------------------

__device__ __forceinline__ float exp_fixed(float x) {
    x = fminf(fmaxf(x, -87.0f), 88.0f);
    const float magic = 12582912.0f;
    float t = __fmul_rn(x, 0x1.715476p+0f);
    float n = __fadd_rn(__fadd_rn(t, magic), -magic);
    float r = __fmaf_rn(n, -0x1.62e4p-1f, x);
    r = __fmaf_rn(n, -0x1.7f7d1cp-20f, r);
    float q = 0x1.a01a02p-13f;
    q = __fmaf_rn(q, r, 0x1.6c16c2p-10f);
    q = __fmaf_rn(q, r, 0x1.111112p-7f);
    q = __fmaf_rn(q, r, 0x1.555556p-5f);
    q = __fmaf_rn(q, r, 0x1.555556p-3f);
    q = __fmaf_rn(q, r, 0.5f);
    q = __fmaf_rn(q, r, 1.0f);
    q = __fmaf_rn(q, r, 1.0f);
    return __fmul_rn(q, __int_as_float(((int)n + 127) << 23));
}

__device__ __forceinline__ float log1p_fixed(float t) {
    float s = __fdiv_rn(t, __fadd_rn(2.0f, t));
    float u = __fmul_rn(s, s);
    float q = 0x1.111112p-4f;
    q = __fmaf_rn(q, u, 0x1.3b13b2p-4f);
    q = __fmaf_rn(q, u, 0x1.745d18p-4f);
    q = __fmaf_rn(q, u, 0x1.c71c72p-4f);
    q = __fmaf_rn(q, u, 0x1.24924ap-3f);
    q = __fmaf_rn(q, u, 0x1.99999ap-3f);
    q = __fmaf_rn(q, u, 0x1.555556p-2f);
    q = __fmaf_rn(q, u, 1.0f);
    return __fmul_rn(__fmul_rn(2.0f, s), q);
}

__device__ __forceinline__ float delta_fixed(float z, float a) {
    float sp = __fadd_rn(fmaxf(z, 0.0f), log1p_fixed(exp_fixed(-fabsf(z))));
    return exp_fixed(__fmul_rn(a, sp));
}

// eight consecutive channels of one value row as fp32
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
    float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
    uint4 a = *reinterpret_cast<const uint4*>(p);
    uint32_t u[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(u[i] << 16);
        v[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
    }
}

// eight consecutive channels of one value row, as loaded (converted to fp32 only when the chain runs)
struct Raw8f { float4 a, b; };
__device__ __forceinline__ Raw8f load_raw8(const float* p) { return {*reinterpret_cast<const float4*>(p), *reinterpret_cast<const float4*>(p + 4)}; }
__device__ __forceinline__ uint4 load_raw8(const __nv_bfloat16* p) { return *reinterpret_cast<const uint4*>(p); }
__device__ __forceinline__ void widen8(const Raw8f& r, float (&v)[8]) {
    v[0] = r.a.x; v[1] = r.a.y; v[2] = r.a.z; v[3] = r.a.w; v[4] = r.b.x; v[5] = r.b.y; v[6] = r.b.z; v[7] = r.b.w;
}
__device__ __forceinline__ void widen8(const uint4& a, float (&v)[8]) {
    const uint32_t u[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(u[i] << 16);
        v[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
    }
}
template <typename T> struct RawOf { using type = uint4; };
template <> struct RawOf<float> { using type = Raw8f; };

// Sum over the LPR lanes of a row group of NB per-lane partials (one per head of a block of NB heads), in the order of the
// xor butterfly (adjacent lanes first: a balanced pairwise tree over the row's 8-channel chunks). The first log2(NB) levels
// are "transposing": a lane keeps half of its values and hands the other half to its partner, so the block costs
// log2(NB) + ... shuffles in all instead of NB log2(LPR) (the additions are the same, and IEEE addition commutes, so the
// bits are those of the plain butterfly). On return p[0] of lane `sub` is the complete sum of head bitrev(sub mod NB) of
// the block (the same value in every lane of the group with those low bits).
template <int NB, int LPR>
__device__ __forceinline__ void block_reduce(float (&p)[NB], int sub) {
    int keep = NB >> 1;
#pragma unroll
    for (int m = 1; m < LPR; m <<= 1) {
        if (keep >= 1) {
            const bool up = (sub & m) != 0;
#pragma unroll
            for (int q = 0; q < NB / 2; ++q) {
                if (q < keep) {
                    const float stay = up ? p[q + keep] : p[q];
                    const float give = up ? p[q] : p[q + keep];
                    p[q] = __fadd_rn(stay, __shfl_xor_sync(0xffffffffu, give, m));
                }
            }
            keep >>= 1;
        } else {
            p[0] = __fadd_rn(p[0], __shfl_xor_sync(0xffffffffu, p[0], m));
        }
    }
}

// One CTA: tiles of kRows consecutive keys of one (batch, KV head), taken in turn with the other CTAs of that pair (grid-
// stride); writes delta for the G query heads of the group. A group of D/8 lanes owns a row: each lane forms the fma chain
// over its 8 channels, an xor butterfly adds adjacent partials pairwise (IEEE addition commutes, so every lane of the group
// holds the same sum). The kernel streams V once and is bound by that stream, so it is built around memory-level
// parallelism: a warp requests ALL value rows of its NEXT tile (kPass 16-byte loads per lane) before it runs the chains of
// the current one, W is staged once per CTA, and softplus / exp of tile t (one (row, head) pair per thread, from the z
// values in shared memory) overlap the chains of tile t + 1 (two z buffers, one barrier per tile).
template <typename T, int D>
__global__ void __launch_bounds__(256, sizeof(T) == 2 ? 2 : 1) delta_kernel(const T* __restrict__ V, const float* __restrict__ W,
                                                    const float* __restrict__ A, float* __restrict__ delta,
                                                    int L, int Hq, int G, int64_t vs_b, int64_t vs_l, int64_t vs_h,
                                                    int j_off, int64_t ld) {
    constexpr int LPR = D / 8;            // lanes per row
    constexpr int RPW = 32 / LPR;         // rows per warp and pass
    constexpr int kRows = 128;
    constexpr int kPass = kRows / (8 * RPW);
    using Raw = typename RawOf<T>::type;
    extern __shared__ float smem[];
    float* sW = smem;                     // [G][D]
    float* sOut = smem + G * D;           // [2][G][kRows]
    const int hk = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LPR, grp = lane / LPR;
    const int ntiles = (L - j_off + kRows - 1) / kRows;        // keys [j_off, L) of a row of ld entries
    const T* Vb = V + b * vs_b + hk * vs_h + sub * 8;
    auto request = [&](int tile, Raw (&raw)[kPass]) {
        const int j0 = j_off + tile * kRows;
#pragma unroll
        for (int t = 0; t < kPass; ++t) {
            const int j = j0 + warp * RPW + grp + t * 8 * RPW;
            if (tile < ntiles && j < L) raw[t] = load_raw8(Vb + (int64_t)j * vs_l);
            else raw[t] = Raw{};
        }
    };
    Raw cur[kPass], nxt[kPass];
    request(blockIdx.x, cur);
    for (int i = tid; i < G * D; i += 256) sW[i] = W[(size_t)hk * G * D + i];
    __syncthreads();
    int buf = 0;
    for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x, buf ^= 1) {
        request(tile + gridDim.x, nxt);
        const int j0 = j_off + tile * kRows, rows = min(kRows, L - j0);
        float* z = sOut + buf * G * kRows;
        // heads in blocks of 4 (then 2, then 1): the chains of a block, then one transposing reduction per pass
        auto block = [&](int g0, auto nb_tag) {
            constexpr int NB = decltype(nb_tag)::value;
            float w[NB][8];
#pragma unroll
            for (int q = 0; q < NB; ++q) {
                const float4 wa = *reinterpret_cast<const float4*>(sW + (g0 + q) * D + sub * 8), wb = *reinterpret_cast<const float4*>(sW + (g0 + q) * D + sub * 8 + 4);
                w[q][0] = wa.x; w[q][1] = wa.y; w[q][2] = wa.z; w[q][3] = wa.w; w[q][4] = wb.x; w[q][5] = wb.y; w[q][6] = wb.z; w[q][7] = wb.w;
            }
            int mine = 0;                 // head of the block this lane ends up with: the low bits of sub, reversed
#pragma unroll
            for (int m = 1, t = NB >> 1; m < NB; m <<= 1, t >>= 1) mine |= (sub & m) ? t : 0;
#pragma unroll
            for (int t = 0; t < kPass; ++t) {
                if (warp * RPW + t * 8 * RPW >= rows) continue;      // (warp-uniform) a short range, e.g. the one appended key of a decoding step
                float v[8], p[NB];
                widen8(cur[t], v);
#pragma unroll
                for (int q = 0; q < NB; ++q) {
                    float a = 0.0f;
#pragma unroll
                    for (int c = 0; c < 8; ++c) a = __fmaf_rn(v[c], w[q][c], a);
                    p[q] = a;
                }
                block_reduce<NB, LPR>(p, sub);
                const int r = warp * RPW + grp + t * 8 * RPW;
                if (sub < NB && r < rows) z[(g0 + mine) * kRows + r] = p[0];
            }
        };
        int g0 = 0;
        for (; g0 + 4 <= G; g0 += 4) block(g0, std::integral_constant<int, 4>{});
        if (g0 + 2 <= G) { block(g0, std::integral_constant<int, 2>{}); g0 += 2; }
        if (g0 < G) block(g0, std::integral_constant<int, 1>{});
        __syncthreads();                  // z of this tile is complete (and the other buffer's readers of two tiles ago are long done)
        for (int i = tid; i < G * kRows; i += 256) {
            const int g = i / kRows, r = i % kRows;
            if (r < rows) delta[((size_t)b * Hq + hk * G + g) * ld + j0 + r] = delta_fixed(z[i], A[hk * G + g]);
        }
#pragma unroll
        for (int t = 0; t < kPass; ++t) cur[t] = nxt[t];
    }
}

// Full sampling weights (Eq. delta_calc as stated: all Hkv*D channels of the value row feed every head's score, the
// linear layer of the App. A listing): z[h] = sum over KV heads hk of (v_hk . W[h, hk*D : (hk+1)*D]), the per-head dot
// products formed as in delta_kernel (8-channel fma chains, pairwise tree over adjacent chunks) and added over hk
// from left to right. One CTA owns 64 keys of one batch and all heads. A group of D/8 lanes owns two rows; it forms the
// chains of D/8 heads at a time and adds them with a transposing butterfly (at each step a lane keeps half of its
// values and hands the other half to its partner: the same additions as the plain butterfly, a quarter of the
// shuffles), after which lane `sub` holds the dot product of head bitrev(sub) and carries that head's running sum.
constexpr int kFullRows = 64;

template <typename T, int D>
__global__ void __launch_bounds__(256) delta_full_kernel(const T* __restrict__ V, const float* __restrict__ W,
                                                         const float* __restrict__ A, float* __restrict__ delta,
                                                         int L, int Hq, int Hkv, int64_t vs_b, int64_t vs_l,
                                                         int64_t vs_h, int j_off, int64_t ld) {
    constexpr int LPR = D / 8;            // lanes per row = heads per batch
    constexpr int RPW = 32 / LPR;         // row groups per warp
    constexpr int kPass = 16 * RPW;       // rows per pass of the CTA (two per lane group)
    extern __shared__ float smem[];
    const int C = Hkv * D, HqP = (Hq + LPR - 1) / LPR * LPR;
    float* sW = smem;                     // [HqP][C], rows beyond Hq zero
    float* sZ = smem + (size_t)HqP * C;   // [HqP][kFullRows]
    const int b = blockIdx.y, j0 = j_off + blockIdx.x * kFullRows;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LPR, grp = lane / LPR;
    int mine = 0;                         // the head (within a batch) this lane ends up with: sub, bit-reversed
#pragma unroll
    for (int m = 1, t = LPR >> 1; m < LPR; m <<= 1, t >>= 1) mine |= (sub & m) ? t : 0;
    for (int i = tid; i < HqP * C; i += 256) sW[i] = i < Hq * C ? W[i] : 0.0f;
    __syncthreads();
    for (int r0 = 0; r0 < kFullRows; r0 += kPass) {
        int r[2];
        r[0] = r0 + warp * 2 * RPW + grp;
        r[1] = r[0] + RPW;
        for (int hk = 0; hk < Hkv; ++hk) {
            float v[2][8];
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                if (j0 + r[n] < L) {
                    load8(V + b * vs_b + (int64_t)(j0 + r[n]) * vs_l + hk * vs_h + sub * 8, v[n]);
                } else {
#pragma unroll
                    for (int c = 0; c < 8; ++c) v[n][c] = 0.0f;
                }
            }
            for (int hb = 0; hb < HqP; hb += LPR) {
                float p[2][LPR];
#pragma unroll
                for (int q = 0; q < LPR; ++q) {
                    const float* wp = sW + (size_t)(hb + q) * C + hk * D + sub * 8;
                    const float4 wa = *reinterpret_cast<const float4*>(wp), wb = *reinterpret_cast<const float4*>(wp + 4);
                    const float w[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
#pragma unroll
                    for (int n = 0; n < 2; ++n) {
                        float a = 0.0f;
#pragma unroll
                        for (int c = 0; c < 8; ++c) a = __fmaf_rn(v[n][c], w[c], a);
                        p[n][q] = a;
                    }
                }
#pragma unroll
                for (int m = 1, keep = LPR >> 1; m < LPR; m <<= 1, keep >>= 1) {
                    const bool up = (sub & m) != 0;
#pragma unroll
                    for (int n = 0; n < 2; ++n)
#pragma unroll
                        for (int q = 0; q < keep; ++q) {
                            const float stay = up ? p[n][q + keep] : p[n][q];
                            const float give = up ? p[n][q] : p[n][q + keep];
                            p[n][q] = __fadd_rn(stay, __shfl_xor_sync(0xffffffffu, give, m));
                        }
                }
                const int h = hb + mine;
#pragma unroll
                for (int n = 0; n < 2; ++n) {
                    float* z = sZ + h * kFullRows + r[n];
                    *z = hk == 0 ? p[n][0] : __fadd_rn(*z, p[n][0]);
                }
            }
        }
    }
    __syncthreads();
    for (int i = tid; i < Hq * kFullRows; i += 256) {
        const int h = i / kFullRows, r = i % kFullRows;
        if (j0 + r < L) delta[((size_t)b * Hq + h) * ld + j0 + r] = delta_fixed(sZ[i], A[h]);
    }
}

// ---- selection --------------------------------------------------------------------------------------------
// Order: key a beats key b iff (delta_a, -a) > (delta_b, -b). delta > 0, so its bit pattern orders like the
// value and one unsigned 64-bit compare decides.
__device__ __forceinline__ unsigned long long sort_key(float dl, int j) {
    return ((unsigned long long)__float_as_uint(dl) << 32) | (unsigned long long)(0xFFFFFFFFu - (unsigned)j);
}

// Chunks are written in DESCENDING order, padding keys (beyond L) carry their index and sort below every real key, and
// the kernel also emits the eight lowest levels of the rank tree (node sizes 256 ... 2, see below) by splitting the sorted
// chunk on one index bit per level.
__global__ void __launch_bounds__(kChunk) chunk_sort_kernel(const float* __restrict__ delta,
                                                            unsigned long long* __restrict__ sorted, int L, int nchunk,
                                                            uint2* __restrict__ lev, int m) {
    __shared__ unsigned long long s[2][kChunk];
    const int bh = blockIdx.y, c = blockIdx.x, t = threadIdx.x, j = c * kChunk + t;
    // padding sorts below every real key (delta > 0) and keeps its index in the low word
    unsigned long long v = j < L ? sort_key(delta[(size_t)bh * L + j], j) : (unsigned long long)(0xFFFFFFFFu - (unsigned)j);
    // bitonic network, ascending; thread t holds position t. Partners less than 32 apart exchange by shuffle, the six
    // wider exchanges go through shared memory (two buffers in turn: one barrier each).
    int nb = 0;
#pragma unroll
    for (int k = 2; k <= kChunk; k <<= 1) {
        const bool up = (t & k) == 0;
#pragma unroll
        for (int mm = k >> 1; mm > 0; mm >>= 1) {
            unsigned long long o;
            if (mm >= 32) {
                s[nb][t] = v;
                __syncthreads();
                o = s[nb][t ^ mm];
                nb ^= 1;
            } else {
                o = __shfl_xor_sync(0xffffffffu, v, mm);
            }
            const bool want_min = ((t & mm) == 0) == up;
            v = want_min ? (v < o ? v : o) : (v > o ? v : o);
        }
    }
    s[0][t] = v;
    __syncthreads();
    const unsigned long long mine = s[0][kChunk - 1 - t];        // position t of the descending order
    sorted[((size_t)bh * nchunk + c) * kChunk + t] = mine;
    // Levels with node size Bs = 256, 128, ..., 2: a node is an aligned block of Bs key indices, its sequence the block's
    // keys in descending order, its bit the half of the block a key lies in. Splitting a node's sequence stably on that
    // bit gives the sequences of its two children.
    __shared__ uint8_t cur[2][kChunk];
    __shared__ uint32_t wbits[kChunk / 32];
    const int lane = t & 31, warp = t >> 5;
    const size_t W = (size_t)nchunk * (kChunk / 32);
    cur[0][t] = (uint8_t)((0xFFFFFFFFu - (uint32_t)mine) & (kChunk - 1));
    __syncthreads();
#pragma unroll
    for (int lv = 0; lv < 8; ++lv) {
        const int Bs = kChunk >> lv, v = cur[lv & 1][t], bit = (v >> (7 - lv)) & 1;
        const uint32_t bal = __ballot_sync(0xffffffffu, bit);
        if (lane == 0) wbits[warp] = bal;
        __syncthreads();
        const int node_start = t & ~(Bs - 1);
        uint32_t cumw = 0;                                      // ones of the node before this word
        for (int k = node_start >> 5; k < warp; ++k) cumw += __popc(wbits[k]);
        const uint32_t below = (1u << lane) - 1u, in_node = Bs >= 32 ? 0xffffffffu : (((1u << Bs) - 1u) << (node_start & 31));
        const int ones_before = (int)cumw + __popc(bal & below & in_node);
        if (lane == 0) lev[((size_t)bh * m + (m - 8 + lv)) * W + (size_t)c * (kChunk / 32) + warp] = make_uint2(cumw, bal);
        const int npos = node_start + (bit ? Bs / 2 + ones_before : (t - node_start) - ones_before);
        cur[(lv + 1) & 1][npos] = (uint8_t)v;
        __syncthreads();
    }
}

// ---- selection as a rank tree -------------------------------------------------------------------------------
// expiry[j] is the w-th smallest INDEX among the keys that beat j, i.e. among the first r entries of the head's keys in
// descending order, r = rank of j. That is a quantile query on a prefix, answered by a tree over key indices: the node of an
// aligned block of 2^k indices stores, for the block's keys in descending order, one bit per key (lower / upper half of
// the block) with running counts. A query walks from the root to a leaf: with c = how many of the first r keys lie in the
// node and z of them in its lower half, the k-th smallest index is in the lower half iff k <= z. log2(L) steps of one
// 8-byte load each, for every key in parallel, whatever w.
// The tree is what a bottom-up merge sort leaves behind: merging the sorted lower and upper half of a block yields the
// block's sorted sequence, and "this output came from the upper half" is the node's bit. chunk_sort_kernel builds the
// levels up to 256 keys; one tree_merge_kernel launch per level does the rest (runs of R keys -> runs of 2R).
// Level l (0 = root) of head bh lives at lev[(bh * m + l) * W + position / 32]: x = ones of the node before this word,
// y = the bits. A trailing run shorter than R (L is not a power of two) merges with what exists; the nodes stay
// left-aligned, which is all a query needs (it never looks past the real keys).
constexpr int kMergeThreads = 256;
constexpr int kMergeOut = 1024;       // outputs per CTA of tree_merge_kernel (four per thread)
constexpr int kBlockKeys = 4096;      // keys one CTA of tree_block_kernel merges in shared memory
constexpr int kBlockThreads = 1024;

// Four consecutive outputs of the merge of two descending runs A (na keys) and B (nb keys), starting at output x:
// i = how many of the first x outputs come from A (the first i for which "A[i] goes before the last B taken" fails), then
// four merge steps. Keys are distinct and non-zero; 0 stands for "run exhausted". Returns i; prov bit u = output u came from B.
__device__ __forceinline__ int merge4(const unsigned long long* A, int na, const unsigned long long* B, int nb, int x,
                                      unsigned long long (&out)[4], uint32_t& prov) {
    int lo = max(0, x - nb), hi = min(x, na);
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (A[mid] > B[x - mid - 1]) lo = mid + 1; else hi = mid;
    }
    int i = lo, k = x - lo;
    unsigned long long a = i < na ? A[i] : 0ull, b = k < nb ? B[k] : 0ull;
    prov = 0u;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const bool takeA = a > b;
        out[u] = takeA ? a : b;
        prov |= takeA ? 0u : 1u << u;
        if (takeA) { ++i; a = i < na ? A[i] : 0ull; } else { ++k; b = k < nb ? B[k] : 0ull; }
    }
    return lo;
}

// the 32-bit word of eight neighbouring threads' four provenance bits each (valid in the lanes with lane % 8 == 0)
__device__ __forceinline__ uint32_t gather_nibbles(uint32_t prov, int lane) {
    uint32_t wv = prov << (4 * (lane & 7));
    wv |= __shfl_xor_sync(0xffffffffu, wv, 1);
    wv |= __shfl_xor_sync(0xffffffffu, wv, 2);
    wv |= __shfl_xor_sync(0xffffffffu, wv, 4);
    return wv;
}

// Levels with nodes of 512 ... 4096 keys in one launch: a CTA holds 4096 keys (16 sorted chunks) in shared memory and
// merges runs of R = 256, 512, 1024, 2048, four consecutive outputs per thread. A node's bit says whether the output came
// from the upper run, and the count of such outputs before a word is the word's position minus the A keys taken so far.
__global__ void __launch_bounds__(kBlockThreads) tree_block_kernel(const unsigned long long* __restrict__ src,
                                                                   unsigned long long* __restrict__ dst,
                                                                   uint2* __restrict__ lev, int Lc, int m) {
    extern __shared__ __align__(16) unsigned long long sk[];         // two buffers of kBlockKeys keys
    const int bh = blockIdx.y, tid = threadIdx.x, lane = tid & 31;
    const int base = blockIdx.x * kBlockKeys, nreal = min(kBlockKeys, Lc - base);
    const size_t Wl = (size_t)Lc / 32;
    unsigned long long* cur = sk;
    unsigned long long* nxt = sk + kBlockKeys;
#pragma unroll
    for (int k = 0; k < kBlockKeys / kBlockThreads; ++k) {
        const int i = tid + k * kBlockThreads;
        cur[i] = i < nreal ? src[(size_t)bh * Lc + base + i] : 0ull;
    }
    __syncthreads();
    const int o = 4 * tid;                                       // this thread's outputs: o .. o + 3 of the block
    int l = m - 9;
    for (int R = kChunk; R < kBlockKeys && R < Lc; R *= 2, --l) {
        const int pair = o & ~(2 * R - 1), x = o - pair;
        const int na = max(0, min(R, nreal - pair)), nb = max(0, min(R, nreal - pair - R));
        unsigned long long out[4];
        uint32_t prov;
        const int i0 = merge4(cur + pair, na, cur + pair + R, nb, x, out, prov);
        const bool exists = o < nreal;                           // (runs are whole chunks: all four outputs exist or none)
        if (exists) {
            *reinterpret_cast<ulonglong2*>(nxt + o) = make_ulonglong2(out[0], out[1]);
            *reinterpret_cast<ulonglong2*>(nxt + o + 2) = make_ulonglong2(out[2], out[3]);
        }
        const uint32_t wv = gather_nibbles(exists ? prov : 0u, lane);
        if ((lane & 7) == 0 && exists) lev[((size_t)bh * m + l) * Wl + (size_t)((base + o) >> 5)] = make_uint2((uint32_t)(x - i0), wv);
        unsigned long long* tmp = cur; cur = nxt; nxt = tmp;
        __syncthreads();
    }
#pragma unroll
    for (int k = 0; k < kBlockKeys / kBlockThreads; ++k) {
        const int i = tid + k * kBlockThreads;
        if (i < nreal) dst[(size_t)bh * Lc + base + i] = cur[i];
    }
}

// One level per launch for runs of R >= 4096 keys: a CTA produces 1024 consecutive outputs of one pair of runs. Warp 0
// finds where they start in the two runs (32 probes per round), the CTA stages up to 1024 keys of each run in shared
// memory, and every thread merges four outputs from there.
__global__ void __launch_bounds__(kMergeThreads) tree_merge_kernel(const unsigned long long* __restrict__ src,
                                                                   unsigned long long* __restrict__ dst,
                                                                   uint2* __restrict__ lev_l, int Lc, int R, int m) {
    __shared__ __align__(16) unsigned long long sA[kMergeOut], sB[kMergeOut];
    __shared__ int s_a0;
    const int bh = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int o0 = blockIdx.x * kMergeOut;                       // first output position of this CTA within the head
    const int base = o0 & ~(2 * R - 1), t0 = o0 - base;
    const int na = min(R, Lc - base), nb = max(0, min(R, Lc - base - R));
    const unsigned long long* A = src + (size_t)bh * Lc + base;
    const unsigned long long* Bv = A + R;
    if (warp == 0) {
        int lo = max(0, t0 - nb), hi = min(t0, na);
        while (lo < hi) {
            const int len = hi - lo, stride = (len + 31) / 32;
            const int i = lo + lane * stride;
            const bool pr = i < hi && A[i] > Bv[t0 - i - 1];      // (i < hi implies i < na and t0 - i > 0)
            const int cnt = __popc(__ballot_sync(0xffffffffu, pr));
            if (cnt == 0) { hi = lo; break; }
            const int last_true = lo + (cnt - 1) * stride;
            lo = last_true + 1;
            hi = min(hi, last_true + stride);
        }
        if (lane == 0) s_a0 = lo;
    }
    __syncthreads();
    const int a0 = s_a0, b0 = t0 - a0;
    const int la = min(kMergeOut, na - a0), lb = min(kMergeOut, nb - b0);
#pragma unroll
    for (int k = 0; k < kMergeOut / kMergeThreads; ++k) {
        const int i = tid + k * kMergeThreads;
        sA[i] = i < la ? A[a0 + i] : 0ull;
        sB[i] = i < lb ? Bv[b0 + i] : 0ull;
    }
    __syncthreads();
    const int x = 4 * tid;
    const bool exists = t0 + x < na + nb;
    unsigned long long out[4];
    uint32_t prov;
    const int i0 = merge4(sA, la, sB, lb, x, out, prov);
    if (exists) {
        unsigned long long* d = dst + (size_t)bh * Lc + o0 + x;
        *reinterpret_cast<ulonglong2*>(d) = make_ulonglong2(out[0], out[1]);
        *reinterpret_cast<ulonglong2*>(d + 2) = make_ulonglong2(out[2], out[3]);
    }
    const uint32_t wv = gather_nibbles(exists ? prov : 0u, lane);
    if ((lane & 7) == 0 && exists) lev_l[(size_t)bh * m * (Lc / 32) + ((o0 + x) >> 5)] = make_uint2((uint32_t)(b0 + x - i0), wv);
}

// One thread per rank r of a head: the key at rank r, the walk down the tree, expiry[j] = max(j, index found).
// kMode 2 (non-causal): every row sees every key, so the key is kept by all rows iff fewer than w keys beat it.
// kMode 1: sequences packed along the key axis (sequence s owns the keys cu[s] <= j < cu[s+1]). A key competes only with
// the keys of its own sequence [s0, s1): of the first r keys of the head, n0 have an index below s0 (a first walk, along
// the path of s0, adds up the lower halves it leaves to its left), so the w-th beater inside the sequence is the
// (n0 + w)-th smallest index overall, if that exists and lies below s1; otherwise the key lives to the end of its sequence.
template <int kMode>
__global__ void __launch_bounds__(256) expiry_tree_kernel(const unsigned long long* __restrict__ sorted, const uint2* __restrict__ lev,
                                                          int32_t* __restrict__ expiry, int L, int Lc, int w, int m,
                                                          const int32_t* __restrict__ cu, int nseq) {
    const int r = blockIdx.x * 256 + threadIdx.x, bh = blockIdx.y;
    if (r >= L) return;                                          // ranks from L on are padding
    const int j = (int)(0xFFFFFFFFu - (uint32_t)sorted[(size_t)bh * Lc + r]);
    const size_t W = (size_t)Lc / 32;
    const uint2* lv0 = lev + (size_t)bh * m * W;
    // ones among the first c entries of the node that starts at position s of a level
    auto ones_of = [](const uint2* lv, int s, int c) {
        const int q = s + c - 1;                                 // last entry of the prefix (c >= 1)
        const uint2 wd = lv[q >> 5];
        const uint32_t upto = (2u << (q & 31)) - 1u, from = ~((1u << (s & 31)) - 1u);         // a node smaller than a word starts inside it
        return (int)wd.x + __popc(wd.y & upto & from);
    };
    int s0 = 0, s1 = L, k = w;
    if (kMode == 1) {
        int lo = 0, hi = nseq;                                   // largest s with cu[s] <= j
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (cu[mid] <= j) lo = mid; else hi = mid;
        }
        s0 = max(cu[lo], 0);
        s1 = min(cu[lo + 1], L);
        if (r >= w && s0 > 0) {
            const uint2* lv = lv0;
            int c = r, s = 0, n0 = 0;
            for (int l = 0; l < m && c > 0; ++l, lv += W) {
                const int half = 1 << (m - 1 - l);
                const int ones = ones_of(lv, s, c);
                if (s0 & half) { n0 += c - ones; c = ones; s += half; } else { c -= ones; }
            }
            k = w + n0;
        }
    }
    int e;
    if (r < k) {
        e = s1;                                                  // fewer than w keys beat it (inside its sequence): never dropped
    } else if (kMode == 2) {
        e = 0;
    } else {
        const uint2* lv = lv0;
        int c = r, s = 0;                                        // k-th smallest among the first c entries of the node starting at s
        for (int l = 0; l < m; ++l, lv += W) {
            const int half = 1 << (m - 1 - l);
            const int ones = ones_of(lv, s, c), zeros = c - ones;
            if (k <= zeros) c = zeros; else { k -= zeros; c = ones; s += half; }
        }
        e = (kMode == 1 && s >= s1) ? s1 : max(j, s);
    }
    expiry[(size_t)bh * L + j] = e;
}

__global__ void fill_i32_kernel(int32_t* p, size_t n, int32_t v) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) p[i] = v;
}

// One CTA per (key tile, head): key j is kept by rows [j, expiry[j]), i.e. by query tiles j/bm .. (expiry[j]-1)/bm.
// A difference array over query tiles forms the union; bits are OR-ed into the (pre-zeroed) bitmap.
// (non-causal mode: key j is kept by rows [0, expiry[j]), so its interval of query tiles starts at tile 0)
__global__ void __launch_bounds__(128) bitmap_kernel(const int32_t* __restrict__ expiry, uint32_t* __restrict__ bitmap,
                                                     int L, int bm, int bn, int Tr, int Wd, int causal) {
    extern __shared__ int diff[];                 // [Tr + 1]
    const int kt = blockIdx.x, bh = blockIdx.y, t = threadIdx.x;
    for (int i = t; i <= Tr; i += blockDim.x) diff[i] = 0;
    __syncthreads();
    const int jend = min(L, (kt + 1) * bn);
    for (int j = kt * bn + t; j < jend; j += blockDim.x) {
        const int e = expiry[(size_t)bh * L + j];
        if (e > (causal ? j : 0)) {
            atomicAdd(&diff[causal ? j / bm : 0], 1);
            atomicAdd(&diff[(e - 1) / bm + 1], -1);
        }
    }
    __syncthreads();
    {   // running sum over the query tiles: each thread owns a contiguous segment, the segment totals are scanned by warp shuffles
        __shared__ int wtot[4];
        const int seg = (Tr + 127) / 128, q0 = t * seg, q1 = min(Tr, q0 + seg);
        int tot = 0;
        for (int q = q0; q < q1; ++q) tot += diff[q];
        int incl = tot;
        const int lane = t & 31, warp = t >> 5;
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += y;
        }
        if (lane == 31) wtot[warp] = incl;
        __syncthreads();
        int run = incl - tot;
        for (int k = 0; k < warp; ++k) run += wtot[k];
        for (int q = q0; q < q1; ++q) { run += diff[q]; diff[q] = run > 0; }
    }
    __syncthreads();
    for (int q = t; q < Tr; q += blockDim.x)
        if (diff[q]) atomicOr(&bitmap[((size_t)bh * Tr + q) * Wd + (kt >> 5)], 1u << (kt & 31));
}

}  // namespace

constexpr int kStaticChunk = kChunk;

// levels of the rank tree over a head of Lc (a multiple of 256) keys: the smallest m with 2^m >= Lc
static int tree_levels(int Lc) {
    int m = 8;
    while ((1ll << m) < Lc) ++m;
    return m;
}

// workspace: header | two buffers of sort keys (8 bytes per padded key each: the merge passes alternate between them) |
// the rank tree (m levels of 8 bytes per 32 padded keys)
size_t mask_ws_bytes(const Prob& P) {
    const size_t nchunk = (P.L + kChunk - 1) / kChunk, keys = (size_t)P.B * P.Hq * nchunk * kChunk;
    return kWsHeaderBytes + keys * 2 * sizeof(unsigned long long) + keys / 32 * tree_levels((int)(nchunk * kChunk)) * sizeof(uint2);
}

template <typename T, int D>
static int launch_delta(const Prob& P, const void* V, const float* W, const float* A, float* bias, cudaStream_t st,
                        int j_begin = 0, int j_end = -1, int64_t ld = -1) {
    if (j_end < 0) j_end = P.L;
    if (ld < 0) ld = P.L;
    if (j_end <= j_begin) return DMA_OK;
    if (P.flags & DMA_FLAG_FULL_DELTA) {
        const size_t HqP = (size_t)(P.Hq + D / 8 - 1) / (D / 8) * (D / 8);
        const size_t bytes = (HqP * P.Hkv * D + HqP * kFullRows) * sizeof(float);
        if (bytes > 200 * 1024) return DMA_ERR_UNSUPPORTED;
        if (cudaFuncSetAttribute(delta_full_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess)
            return DMA_ERR_CUDA;
        delta_full_kernel<T, D><<<dim3((j_end - j_begin + kFullRows - 1) / kFullRows, P.B), 256, bytes, st>>>(
            (const T*)V, W, A, bias, j_end, P.Hq, P.Hkv, P.vs[0], P.vs[1], P.vs[2], j_begin, ld);
        count_launch();
        return check_launch();
    }
    // two CTAs per SM in all (what the register file holds at once), each walking its (batch, KV head) pair's tiles grid-stride; short ranges (one appended key
    // of a decoding step) get one CTA per tile
    const int ntiles = (j_end - j_begin + 127) / 128;
    int per_pair = (2 * 148 + P.Hkv * P.B - 1) / (P.Hkv * P.B);
    per_pair = per_pair < 1 ? 1 : per_pair > ntiles ? ntiles : per_pair;
    dim3 grid(per_pair, P.Hkv, P.B);
    size_t smem = (size_t)P.G * (D + 2 * 128) * sizeof(float);
    if (smem > 48 * 1024) return DMA_ERR_UNSUPPORTED;
    delta_kernel<T, D><<<grid, 256, smem, st>>>((const T*)V, W, A, bias, j_end, P.Hq, P.G, P.vs[0], P.vs[1], P.vs[2], j_begin, ld);
    count_launch();
    return check_launch();
}

// delta for the keys [j_begin, j_end) only, into rows of ld entries (a decoding cache that grows)
int launch_delta_range(const Prob& P, const void* V, const float* W, const float* A, float* delta, int64_t ld, int j_begin,
                       int j_end, cudaStream_t st) {
    if (P.dtype == DMA_BF16)
        return P.d == 128 ? launch_delta<__nv_bfloat16, 128>(P, V, W, A, delta, st, j_begin, j_end, ld)
                          : launch_delta<__nv_bfloat16, 64>(P, V, W, A, delta, st, j_begin, j_end, ld);
    return P.d == 128 ? launch_delta<float, 128>(P, V, W, A, delta, st, j_begin, j_end, ld)
                      : launch_delta<float, 64>(P, V, W, A, delta, st, j_begin, j_end, ld);
}

// size limits of the stage's kernels (shared-memory footprints), checked before anything is enqueued
static int mask_build_limits(const Prob& P) {
    if (P.flags & DMA_FLAG_FULL_DELTA) {
        const size_t lanes = (size_t)P.d / 8, HqP = (P.Hq + lanes - 1) / lanes * lanes;
        if ((HqP * P.Hkv * P.d + HqP * kFullRows) * sizeof(float) > 200 * 1024) return DMA_ERR_UNSUPPORTED;
    } else if ((size_t)P.G * (P.d + 2 * 128) * sizeof(float) > 48 * 1024) {
        return DMA_ERR_UNSUPPORTED;
    }
    if ((size_t)(P.Tr + 1) * sizeof(int) > 48 * 1024) return DMA_ERR_UNSUPPORTED;
    return DMA_OK;
}

int launch_mask_build(const Prob& P, const void* V, const float* W, const float* A, float* bias, int32_t* expiry,
                      uint32_t* bitmap, void* ws, cudaStream_t st, const int32_t* cu, int nseq) {
    int rc;
    if ((rc = mask_build_limits(P))) return rc;          // an error return means that no kernel has been launched
    constexpr size_t kBlockSmem = 2 * (size_t)kBlockKeys * sizeof(unsigned long long);
    if (cudaFuncSetAttribute(tree_block_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBlockSmem) != cudaSuccess) return DMA_ERR_CUDA;
    if (P.dtype == DMA_BF16)
        rc = P.d == 128 ? launch_delta<__nv_bfloat16, 128>(P, V, W, A, bias, st)
                        : launch_delta<__nv_bfloat16, 64>(P, V, W, A, bias, st);
    else
        rc = P.d == 128 ? launch_delta<float, 128>(P, V, W, A, bias, st) : launch_delta<float, 64>(P, V, W, A, bias, st);
    if (rc) return rc;

    const int BH = P.B * P.Hq;
    const int nchunk = (P.L + kChunk - 1) / kChunk;
    if (P.w >= P.L && !cu) {   // every visible key is kept
        size_t n = (size_t)BH * P.L;
        fill_i32_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(expiry, n, P.L);
        count_launch();
    } else {
        // rank tree: sorted chunks and the low levels, one merge pass per further level, then one walk per key
        const int Lc = nchunk * kChunk, m = tree_levels(Lc);
        const size_t keys = (size_t)BH * Lc, Wl = (size_t)Lc / 32;
        auto* buf0 = reinterpret_cast<unsigned long long*>((char*)ws + kWsHeaderBytes);
        auto* buf1 = buf0 + keys;
        uint2* lev = reinterpret_cast<uint2*>(buf1 + keys);
        chunk_sort_kernel<<<dim3(nchunk, BH), kChunk, 0, st>>>(bias, buf0, P.L, nchunk, lev, m);
        int launches = 2;
        if (Lc > kChunk) {
            tree_block_kernel<<<dim3((Lc + kBlockKeys - 1) / kBlockKeys, BH), kBlockThreads, kBlockSmem, st>>>(buf0, buf1, lev, Lc, m);
            std::swap(buf0, buf1);
            ++launches;
        }
        int l = m - 13;                                          // level of the nodes of 2 * kBlockKeys keys
        for (int R = kBlockKeys; R < Lc; R *= 2, --l, ++launches) {
            tree_merge_kernel<<<dim3((Lc + kMergeOut - 1) / kMergeOut, BH), kMergeThreads, 0, st>>>(buf0, buf1, lev + (size_t)l * Wl, Lc, R, m);
            std::swap(buf0, buf1);
        }
        const dim3 grid((P.L + 255) / 256, BH);
        if (cu) expiry_tree_kernel<1><<<grid, 256, 0, st>>>(buf0, lev, expiry, P.L, Lc, P.w, m, cu, nseq);
        else if (P.causal) expiry_tree_kernel<0><<<grid, 256, 0, st>>>(buf0, lev, expiry, P.L, Lc, P.w, m, nullptr, 0);
        else expiry_tree_kernel<2><<<grid, 256, 0, st>>>(buf0, lev, expiry, P.L, Lc, P.w, m, nullptr, 0);
        count_launch(launches);
    }
    if ((rc = check_launch())) return rc;

    if (cudaMemsetAsync(bitmap, 0, (size_t)BH * P.Tr * P.Wd * sizeof(uint32_t), st) != cudaSuccess) return DMA_ERR_CUDA;
    size_t smem = (size_t)(P.Tr + 1) * sizeof(int);
    if (smem > 48 * 1024) return DMA_ERR_UNSUPPORTED;
    bitmap_kernel<<<dim3(P.Tc, BH), 128, smem, st>>>(expiry, bitmap, P.L, P.bm, P.bn, P.Tr, P.Wd, P.causal);
    count_launch();
    return check_launch();
}

}  // namespace dma

// ---------------------------------------------------------------------------------------------------------------
// dma_mask_build_static: mask generation for callers that cannot hand over a workspace.
// The selection's scratch (sort keys and rank tree) lives in this file-scope device array, which every GPU that loads the library keeps
// until the process exits. In host code the array's name is only a stand-in; its device address is looked up
// once per device with cudaGetSymbolAddress and that pointer is what the kernels receive.
// ---------------------------------------------------------------------------------------------------------------
namespace {
// 1 Mi padded keys: two buffers of sort keys (8 MiB each) and a rank tree of at most 20 levels (8 bytes per 32 keys and
// level: 5 MiB). B * Hq * roundup(L, 256) must not exceed this.
constexpr size_t kStaticKeys = 1u << 20;
static __device__ __align__(256) unsigned long long g_static_scratch[dma::kWsHeaderBytes / 8 + 2 * kStaticKeys + kStaticKeys / 32 * 20];
constexpr int kMaxDevices = 64;
void* g_static_ptr[kMaxDevices];            // per-device address of g_static_scratch (0 = not looked up yet)
std::mutex g_static_mutex;
}  // namespace

extern "C" int dma_mask_build_static(const dma_problem_t* p, const void* V, const float* W_delta, const float* A,
                                     float* bias, int32_t* expiry, uint32_t* bitmap, void* cuda_stream) {
    dma::Prob P;
    int rc = dma::resolve(p, &P);
    if (rc) return rc;
    if (!V || !W_delta || !A || !bias || !expiry || !bitmap) return DMA_ERR_NULL;
    const uintptr_t bits = (uintptr_t)V | (uintptr_t)W_delta | (uintptr_t)bias | (uintptr_t)expiry | (uintptr_t)bitmap;
    if (bits & 15) return DMA_ERR_ALIGN;
    const size_t keys = (size_t)P.B * P.Hq * ((P.L + dma::kStaticChunk - 1) / dma::kStaticChunk) * dma::kStaticChunk;
    if (keys > kStaticKeys) return DMA_ERR_WORKSPACE;          // larger problems must use dma_mask_build
    int dev = -1, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DMA_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess || major != 10) return DMA_ERR_CUDA;
    void* scratch;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ptr[dev]) {       // first call on this device (which is current): resolve the symbol's address
            void* ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return DMA_ERR_CUDA;
            g_static_ptr[dev] = ptr;
        }
        scratch = g_static_ptr[dev];
    }
    return dma::launch_mask_build(P, V, W_delta, A, bias, expiry, bitmap, scratch, (cudaStream_t)cuda_stream);
}
