// Decoding step (Sec. 3.2 for a single query at the end of the sequence; Alg. 1 with the per-key mask M in R^N, the
// configuration of the paper's decode benchmark): every (batch, query head) keeps the w cached keys with the largest
// dynamic weight delta (ties to the lower index; all N keys if N <= w) and attends to them with delta as the bias.
// HBM / L2-bound: the delta row is scanned to select, then only the selected K and V rows are read.
//
// Kernels
//   decode_row_select_kernel   rows of up to 32768 keys: radix select over the 64-bit keys (delta bits << 32 | ~index) for
//                          the threshold T with exactly min(w, N) keys >= T, one CTA per row on a shared-memory copy of the
//                          row (a decoding step at these lengths is bound by dependent launches, not by their work)
//   decode_hist_kernel x3, decode_thr_kernel   longer rows: the same three histogram passes spread over CTAs of 8192 keys
//                          (per-row global histograms) and the final pick
//   decode_index_kernel    optional: the selected indices in ascending order
//   decode_attn_kernel     per (batch, head, split of <= 2048 keys): selected keys of the split are compacted into shared
//                          memory; each warp then takes four of them per round (8 bytes of the K / V row per lane),
//                          online softmax per warp, warps combined in shared memory -> partial (m, l, o). The CTA that
//                          finishes a row last (a ticket counter, no waiting) combines the row's partials -> o, log-sum-exp
#include "common.cuh"

namespace dma {
namespace {

constexpr int kSplitKeys = 2048;
constexpr int kAttnThreads = 256;

__device__ __forceinline__ unsigned long long key_of(float dl, int j) {
    return ((unsigned long long)__float_as_uint(dl) << 32) | (unsigned long long)(0xFFFFFFFFu - (unsigned)j);
}

// Radix select of the min(w, N)-th largest key of every (batch, head) row, spread over many CTAs. Three histogram
// passes over the delta bit patterns, bits [30:20], [19:9], [8:0] (delta > 0: the sign bit is clear and the pattern orders
// like the value; exponent plus three mantissa bits spread a row over enough bins that shared-memory adds rarely
// collide). Pass p: every CTA first re-derives the prefix chosen by the passes before it from their global histograms
// (pick_bin: a 2048-bin suffix scan, identical in every CTA), then histograms the next bits of its 8192-key slice of the
// row for the keys that match the prefix and adds the non-zero bins to the row's global histogram. A last kernel picks
// the final bin and, only if several keys tie at the threshold delta and not all of them are wanted, walks the row in
// index order for the cut. state[bh] = {prefix bits, keys still wanted inside the prefix}.
struct SelState { uint32_t prefix; int need; };

// hist: 2048 counters of one pass; returns through `st` the bin holding the need-th largest key (scanning from the top
// bin) and the rank wanted inside it. Called by every thread of a CTA of 256 threads.
__device__ __forceinline__ void pick_bin(const int* __restrict__ hist, int shift, SelState& st, int* s_scan, SelState* s_out) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int c[8], sum = 0;
#pragma unroll
    for (int t = 0; t < 8; ++t) { c[t] = __ldcg(&hist[2047 - (8 * tid + t)]); sum += c[t]; }       // descending bin order
    int incl = sum;
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    int before = 0;
    for (int wq = 0; wq < warp; ++wq) before += s_scan[wq];
    int excl = before + incl - sum;                       // keys in bins above this thread's first bin
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        if (excl < st.need && st.need <= excl + c[t]) {
            s_out->prefix = st.prefix | ((uint32_t)(2047 - (8 * tid + t)) << shift);
            s_out->need = st.need - excl;
        }
        excl += c[t];
    }
    __syncthreads();
    st = *s_out;
    __syncthreads();
}

constexpr int kSliceKeys = 8192;

// one histogram pass (pass = 0, 1, 2) of one 8192-key slice of one row; ghist [3][BH][2048] zeroed before pass 0
__device__ __forceinline__ void hist_slice(const float* __restrict__ delta, int64_t ld, int N, int w, int pass, int* __restrict__ ghist,
                                           int BH, int bh, int slice, int* hist, int* s_scan, SelState* s_out_p) {
    SelState& s_out = *s_out_p;
    const int tid = threadIdx.x;
    const float* dl = delta + (size_t)bh * ld;
    const int shifts[3] = {20, 9, 0}, widths[3] = {11, 11, 9};
    SelState st{0u, w};
    for (int q = 0; q < pass; ++q) pick_bin(ghist + ((size_t)q * BH + bh) * 2048, shifts[q], st, s_scan, &s_out);
    for (int t = tid; t < 2048; t += 256) hist[t] = 0;
    __syncthreads();
    const int shift = shifts[pass], nb = 1 << widths[pass];
    const uint32_t himask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + widths[pass]));
    const int j0 = slice * kSliceKeys, j1 = min(N, j0 + kSliceKeys);
    for (int base = j0; base < j1; base += 4 * 256) {
        uint32_t u[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const int j = base + t * 256 + tid;
            u[t] = j < j1 ? __float_as_uint(dl[j]) : 0xFFFFFFFFu;              // never matches: deltas have the sign bit clear
        }
#pragma unroll
        for (int t = 0; t < 4; ++t)
            if (u[t] != 0xFFFFFFFFu && (u[t] & himask) == st.prefix) atomicAdd(&hist[(u[t] >> shift) & (nb - 1)], 1);
    }
    __syncthreads();
    int* g = ghist + ((size_t)pass * BH + bh) * 2048;
    for (int t = tid; t < 2048; t += 256)
        if (hist[t]) atomicAdd(&g[t], hist[t]);
    __syncthreads();                               // the shared histogram is reused by the caller's next slice
}

__global__ void __launch_bounds__(256) decode_hist_kernel(const float* __restrict__ delta, int64_t ld, int N, int w, int pass,
                                                          int* __restrict__ ghist, int BH) {
    __shared__ int hist[2048];
    __shared__ int s_scan[8];
    __shared__ SelState s_out;
    if (N <= w) return;
    hist_slice(delta, ld, N, w, pass, ghist, BH, blockIdx.y, blockIdx.x, hist, s_scan, &s_out);
}

// one CTA per row: final pick; thr = (delta bits << 32) | ~index cut
__device__ __forceinline__ void thr_row(const float* __restrict__ delta, int64_t ld, int N, int w, const int* __restrict__ ghist, int BH,
                                        unsigned long long* __restrict__ thr, int bh, int* s_scan, SelState* s_out_p, int* s_warp,
                                        int* s_found_p) {
    SelState& s_out = *s_out_p;
    int& s_found = *s_found_p;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (N <= w) {
        if (tid == 0) thr[bh] = 0ull;          // every key qualifies
        return;
    }
    const float* dl = delta + (size_t)bh * ld;
    const int shifts[3] = {20, 9, 0};
    SelState st{0u, w};
    const int* g2 = ghist + ((size_t)2 * BH + bh) * 2048;
    for (int q = 0; q < 3; ++q) pick_bin(ghist + ((size_t)q * BH + bh) * 2048, shifts[q], st, s_scan, &s_out);
    // st.prefix = delta bits of the threshold; st.need of the keys with exactly that delta are kept, lowest index first
    const uint32_t dstar = st.prefix;
    const int equal = __ldcg(&g2[dstar & 511]);
    if (st.need >= equal) {                    // every key with this delta is wanted: no cut inside the group
        if (tid == 0) thr[bh] = (unsigned long long)dstar << 32;
        return;
    }
    if (tid == 0) s_found = -1;
    int seen = 0;
    for (int base = 0; base < N; base += 256) {
        const int j = base + tid;
        const bool eq = j < N && __float_as_uint(dl[j]) == dstar;
        const uint32_t bal = __ballot_sync(0xffffffffu, eq);
        if (lane == 0) s_warp[warp] = __popc(bal);
        __syncthreads();
        int before = 0, total = 0;
#pragma unroll
        for (int wq = 0; wq < 8; ++wq) {
            const int c = s_warp[wq];
            before += wq < warp ? c : 0;
            total += c;
        }
        const int rank = seen + before + __popc(bal & ((1u << lane) - 1));      // 0-based rank among the equal keys
        if (eq && rank == st.need - 1) s_found = j;
        seen += total;
        __syncthreads();
        if (seen >= st.need) break;
    }
    __syncthreads();
    if (tid == 0) thr[bh] = key_of(__uint_as_float(dstar), s_found);
}

__global__ void __launch_bounds__(256) decode_thr_kernel(const float* __restrict__ delta, int64_t ld, int N, int w,
                                                         const int* __restrict__ ghist, int BH, unsigned long long* __restrict__ thr) {
    __shared__ int s_scan[8];
    __shared__ SelState s_out;
    __shared__ int s_warp[8], s_found;
    thr_row(delta, ld, N, w, ghist, BH, thr, blockIdx.x, s_scan, &s_out, s_warp, &s_found);
}

// The whole selection of a row by ONE CTA, for rows that fit in shared memory (N <= kRowSelectMax): the row is loaded
// once, the three histogram passes and the final pick run on the shared copy with CTA-wide barriers only. A decoding step
// at these lengths is bound by dependent launches and global round trips, not by the work: this replaces a memset and
// four launches by one. Also zeroes the row's combine ticket.
constexpr int kRowSelectMax = 32768;
constexpr int kRowSelectThreads = 1024;

__global__ void __launch_bounds__(kRowSelectThreads) decode_row_select_kernel(const float* __restrict__ delta, int64_t ld, int N, int w,
                                                                              unsigned long long* __restrict__ thr, int* __restrict__ tickets) {
    extern __shared__ uint32_t row[];                  // the row's delta bit patterns
    __shared__ int hist[2048];
    __shared__ int s_scan[32];
    __shared__ uint32_t s_prefix;
    __shared__ int s_need, s_equal, s_found, s_warp[32];
    const int bh = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) tickets[bh] = 0;
    if (N <= w) {
        if (tid == 0) thr[bh] = 0ull;                  // every key qualifies
        return;
    }
    const float* dl = delta + (size_t)bh * ld;
    for (int j = tid; j < N; j += kRowSelectThreads) row[j] = __float_as_uint(dl[j]);
    uint32_t prefix = 0u;
    int need = w;
    const int shifts[3] = {20, 9, 0}, widths[3] = {11, 11, 9};
    for (int pass = 0; pass < 3; ++pass) {
        for (int t = tid; t < 2048; t += kRowSelectThreads) hist[t] = 0;
        __syncthreads();                               // (also: the row is complete before the first pass reads it)
        const int shift = shifts[pass], nb = 1 << widths[pass];
        const uint32_t himask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + widths[pass]));
        for (int j = tid; j < N; j += kRowSelectThreads) {
            const uint32_t u = row[j];
            if ((u & himask) == prefix) atomicAdd(&hist[(u >> shift) & (nb - 1)], 1);
        }
        __syncthreads();
        // the bin holding the need-th largest key, scanning from the top bin: two bins per thread, descending order
        const int c0 = hist[2047 - 2 * tid], c1 = hist[2046 - 2 * tid], sum = c0 + c1;
        int incl = sum;
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) s_scan[warp] = incl;
        __syncthreads();
        int before = 0;
        for (int wq = 0; wq < warp; ++wq) before += s_scan[wq];
        int excl = before + incl - sum;                // keys in bins above this thread's first bin
        if (excl < need && need <= excl + c0) { s_prefix = prefix | ((uint32_t)(2047 - 2 * tid) << shift); s_need = need - excl; s_equal = c0; }
        excl += c0;
        if (excl < need && need <= excl + c1) { s_prefix = prefix | ((uint32_t)(2046 - 2 * tid) << shift); s_need = need - excl; s_equal = c1; }
        __syncthreads();
        prefix = s_prefix;
        need = s_need;
        __syncthreads();
    }
    // prefix = delta bits of the threshold; `need` of the keys with exactly that delta are kept, lowest index first
    const int equal = s_equal;
    if (need >= equal) {                               // every key with this delta is wanted: no cut inside the group
        if (tid == 0) thr[bh] = (unsigned long long)prefix << 32;
        return;
    }
    if (tid == 0) s_found = -1;
    int seen = 0;
    for (int base = 0; base < N; base += kRowSelectThreads) {
        const int j = base + tid;
        const bool eq = j < N && row[j] == prefix;
        const uint32_t bal = __ballot_sync(0xffffffffu, eq);
        if (lane == 0) s_warp[warp] = __popc(bal);
        __syncthreads();
        int bef = 0, total = 0;
        for (int wq = 0; wq < 32; ++wq) {
            const int c = s_warp[wq];
            bef += wq < warp ? c : 0;
            total += c;
        }
        const int rank = seen + bef + __popc(bal & ((1u << lane) - 1));          // 0-based rank among the equal keys
        if (eq && rank == need - 1) s_found = j;
        seen += total;
        __syncthreads();
        if (seen >= need) break;
    }
    __syncthreads();
    if (tid == 0) thr[bh] = key_of(__uint_as_float(prefix), s_found);
}

__global__ void __launch_bounds__(256) decode_index_kernel(const float* __restrict__ delta, int64_t ld, int N, int keep,
                                                           const unsigned long long* __restrict__ thr, int32_t* __restrict__ idx,
                                                           int64_t idx_stride) {
    __shared__ int wsum[2][8];
    const int bh = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* dl = delta + (size_t)bh * ld;
    const unsigned long long T = thr[bh];
    int n = 0, buf = 0;
    for (int base = 0; base < N; base += 256, buf ^= 1) {
        const int j = base + tid;
        const bool sel = j < N && key_of(dl[j], j) >= T;
        const uint32_t bal = __ballot_sync(0xffffffffu, sel);
        if (lane == 0) wsum[buf][warp] = __popc(bal);
        __syncthreads();
        int before = 0, total = 0;
#pragma unroll
        for (int wq = 0; wq < 8; ++wq) {
            const int c = wsum[buf][wq];
            before += wq < warp ? c : 0;
            total += c;
        }
        const int pos = n + before + __popc(bal & ((1u << lane) - 1));
        if (sel && pos < keep) idx[(size_t)bh * idx_stride + pos] = j;
        n += total;
    }
}

__device__ __forceinline__ void load4(const float* p, float (&v)[4]) {
    const float4 a = *reinterpret_cast<const float4*>(p);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16* p, float (&v)[4]) {
    const uint2 a = *reinterpret_cast<const uint2*>(p);
    v[0] = __uint_as_float(a.x << 16); v[1] = __uint_as_float(a.x & 0xffff0000u);
    v[2] = __uint_as_float(a.y << 16); v[3] = __uint_as_float(a.y & 0xffff0000u);
}

// partial [bh][split][D + 2]: o (unnormalised, relative to m), m (log2 domain), l
// The attention part shared by the two decoding kernels: `list` (shared memory) holds `count` key indices of this CTA.
// Each warp takes four of them per round (8 bytes of the K / V row per lane), online softmax per warp, then the warps are
// combined in shared memory and the CTA's partial (o relative to m, m in the log2 domain, l) is written.
template <typename T, int D>
__device__ __forceinline__ void decode_attend(const int* list, int count, const T* __restrict__ q, const T* __restrict__ K,
                                              const T* __restrict__ V, const float* __restrict__ dl, float* __restrict__ out,
                                              int bh, int b, int hk, float scale_log2, int64_t ks_b, int64_t ks_l, int64_t ks_h,
                                              int64_t vs_b, int64_t vs_l, int64_t vs_h) {
    constexpr int LPK = D / 4;                 // lanes per key row (4 channels per lane)
    constexpr int KPW = 32 / LPK;              // keys per warp instruction
    __shared__ float s_part[8][D + 2];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // each warp: KPW keys per instruction (LPK lanes per key, 4 channels per lane), four such groups per round
    const int sub = lane % LPK, grp = lane / LPK;
    float qv[4];
    load4(q + (size_t)bh * D + sub * 4, qv);
    float m = -INFINITY, l = 0.0f, o[4] = {0.f, 0.f, 0.f, 0.f};
    const T* Kb = K + b * ks_b + hk * ks_h + sub * 4;
    const T* Vb = V + b * vs_b + hk * vs_h + sub * 4;
    constexpr int kInFlight = 4;               // key rows whose K and V loads are in flight together, per lane group (8 was slower)
    for (int base = warp * KPW * kInFlight; base < count; base += 8 * KPW * kInFlight) {
        int jj[kInFlight];
        float kv[kInFlight][4], vv[kInFlight][4], bias[kInFlight];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            const int e = base + u * KPW + grp;
            jj[u] = e < count ? list[e] : -1;
            if (jj[u] >= 0) {
                load4(Kb + (int64_t)jj[u] * ks_l, kv[u]);
                load4(Vb + (int64_t)jj[u] * vs_l, vv[u]);
                bias[u] = dl[jj[u]];
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c) { kv[u][c] = 0.0f; vv[u][c] = 0.0f; }
                bias[u] = 0.0f;
            }
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            float s = qv[0] * kv[u][0] + qv[1] * kv[u][1] + qv[2] * kv[u][2] + qv[3] * kv[u][3];
#pragma unroll
            for (int mm = 1; mm < LPK; mm <<= 1) s += __shfl_xor_sync(0xffffffffu, s, mm);
            const float x = jj[u] >= 0 ? fmaf(s, scale_log2, bias[u] * 1.4426950408889634f) : -INFINITY;
            const float m_new = fmaxf(m, x);
            const float f = m_new == -INFINITY ? 1.0f : exp2f(m - m_new);
            const float p = m_new == -INFINITY ? 0.0f : exp2f(x - m_new);
            l = l * f + p;
#pragma unroll
            for (int c = 0; c < 4; ++c) o[c] = o[c] * f + p * vv[u][c];
            m = m_new;
        }
    }
    // the KPW key groups of a warp hold different keys: merge them, then the warps, in shared memory
#pragma unroll
    for (int mm = LPK; mm < 32; mm <<= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, mm), l2 = __shfl_xor_sync(0xffffffffu, l, mm);
        float o2[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) o2[c] = __shfl_xor_sync(0xffffffffu, o[c], mm);
        const float mn = fmaxf(m, m2);
        const float f1 = mn == -INFINITY ? 1.0f : exp2f(m - mn), f2 = mn == -INFINITY ? 1.0f : exp2f(m2 - mn);
        l = l * f1 + l2 * f2;
#pragma unroll
        for (int c = 0; c < 4; ++c) o[c] = o[c] * f1 + o2[c] * f2;
        m = mn;
    }
    if (grp == 0) {
#pragma unroll
        for (int c = 0; c < 4; ++c) s_part[warp][sub * 4 + c] = o[c];
        if (sub == 0) { s_part[warp][D] = m; s_part[warp][D + 1] = l; }
    }
    __syncthreads();
    float mx = -INFINITY;
#pragma unroll
    for (int wq = 0; wq < 8; ++wq) mx = fmaxf(mx, s_part[wq][D]);
    for (int c = tid; c < D + 2; c += kAttnThreads) {
        if (c == D) { out[c] = mx; continue; }
        float acc = 0.0f;
#pragma unroll
        for (int wq = 0; wq < 8; ++wq) {
            const float mw = s_part[wq][D];
            const float f = (mw == -INFINITY || mx == -INFINITY) ? 0.0f : exp2f(mw - mx);
            acc += s_part[wq][c] * f;                 // c == D + 1 is l
        }
        out[c] = acc;
    }
}

// The row's partials -> o, log-sum-exp; every thread of a 256-thread CTA takes part: warp g takes the splits s = g, g + 8, ...
// with D / 32 channels per lane, then the eight warps are merged in shared memory. The partials come from other CTAs: read at L2.
template <typename T, int D>
__device__ __forceinline__ void combine_row(const float* __restrict__ partial, T* __restrict__ o, float* __restrict__ lse, int nsplit, int bh) {
    constexpr int CPL = D / 32;                // channels per lane
    __shared__ float s_m[8], s_l[8], s_o[8][D];
    const int lane = threadIdx.x & 31, g = threadIdx.x >> 5;
    const float* p = partial + (size_t)bh * nsplit * (D + 2);
    float mx = -INFINITY;
    for (int s = g; s < nsplit; s += 8) mx = fmaxf(mx, __ldcg(&p[(size_t)s * (D + 2) + D]));
    float l = 0.0f, acc[CPL];
#pragma unroll
    for (int c = 0; c < CPL; ++c) acc[c] = 0.0f;
    for (int s = g; s < nsplit; s += 8) {
        const float* ps = p + (size_t)s * (D + 2);
        const float ms = __ldcg(&ps[D]);
        const float f = ms == -INFINITY ? 0.0f : exp2f(ms - mx);
        l += __ldcg(&ps[D + 1]) * f;
#pragma unroll
        for (int c = 0; c < CPL; ++c) acc[c] += __ldcg(&ps[lane * CPL + c]) * f;
    }
#pragma unroll
    for (int c = 0; c < CPL; ++c) s_o[g][lane * CPL + c] = acc[c];
    if (lane == 0) { s_m[g] = mx; s_l[g] = l; }
    __syncthreads();
    if (threadIdx.x < D) {
        const int c = threadIdx.x;
        float m_all = -INFINITY;
#pragma unroll
        for (int q = 0; q < 8; ++q) m_all = fmaxf(m_all, s_m[q]);
        float lt = 0.0f, at = 0.0f;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float f = s_m[q] == -INFINITY ? 0.0f : exp2f(s_m[q] - m_all);
            lt += s_l[q] * f;
            at += s_o[q][c] * f;
        }
        const float v = lt > 0.0f ? at / lt : 0.0f;
        if constexpr (sizeof(T) == 2) o[(size_t)bh * D + c] = __float2bfloat16_rn(v); else o[(size_t)bh * D + c] = v;
        if (c == 0) lse[bh] = lt > 0.0f ? 0.6931471805599453f * (m_all + log2f(lt)) : -INFINITY;
    }
}

// Called by every thread of an attention CTA after its partial is written: the CTA that finishes its row last (a ticket
// counter, which it resets for the next call; nobody waits) combines the row. Returns true in that CTA.
__device__ __forceinline__ bool last_of_row(int* ticket, int nsplit) {
    __shared__ int s_last;
    __syncthreads();                                   // every thread's part of the partial is written ...
    if (threadIdx.x == 0) {
        __threadfence();                               // ... and visible device-wide before the ticket is taken (the fence is cumulative)
        const int t = atomicAdd(ticket, 1);
        s_last = t == nsplit - 1;
        if (s_last) {
            *ticket = 0;
            __threadfence();                           // the other CTAs' partials, published before their tickets, are visible from here on
        }
    }
    __syncthreads();
    return s_last != 0;
}

template <typename T, int D>
__global__ void __launch_bounds__(kAttnThreads) decode_attn_kernel(const T* __restrict__ q, const T* __restrict__ K, const T* __restrict__ V,
                                                                   const float* __restrict__ delta, int64_t ld,
                                                                   const unsigned long long* __restrict__ thr, float* __restrict__ partial,
                                                                   int N, int Hq, int G, float scale_log2, int nsplit,
                                                                   int64_t ks_b, int64_t ks_l, int64_t ks_h, int64_t vs_b, int64_t vs_l,
                                                                   int64_t vs_h, int* __restrict__ tickets, T* __restrict__ o,
                                                                   float* __restrict__ lse) {
    __shared__ int list[kSplitKeys];
    __shared__ int s_count, wsum[2][8];
    const int split = blockIdx.x, bh = blockIdx.y, b = bh / Hq, h = bh % Hq, hk = h / G;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* dl = delta + (size_t)bh * ld;
    const unsigned long long Tkey = thr[bh];
    const int j_begin = split * kSplitKeys, j_end = min(N, j_begin + kSplitKeys);
    // ordered compaction of the split's selected keys
    int n = 0, buf = 0;
    float dpre[kSplitKeys / kAttnThreads];          // the split's deltas of this thread, all loads in flight together
#pragma unroll
    for (int t = 0; t < kSplitKeys / kAttnThreads; ++t) {
        const int j = j_begin + t * kAttnThreads + tid;
        dpre[t] = j < j_end ? dl[j] : 0.0f;
    }
#pragma unroll
    for (int t = 0; t < kSplitKeys / kAttnThreads; ++t, buf ^= 1) {
        const int base = j_begin + t * kAttnThreads;
        if (base >= j_end) break;
        const int j = base + tid;
        const bool sel = j < j_end && key_of(dpre[t], j) >= Tkey;
        const uint32_t bal = __ballot_sync(0xffffffffu, sel);
        if (lane == 0) wsum[buf][warp] = __popc(bal);
        __syncthreads();
        int before = 0, total = 0;
#pragma unroll
        for (int wq = 0; wq < 8; ++wq) {
            const int c = wsum[buf][wq];
            before += wq < warp ? c : 0;
            total += c;
        }
        if (sel) list[n + before + __popc(bal & ((1u << lane) - 1))] = j;
        n += total;
    }
    if (tid == 0) s_count = n;
    __syncthreads();
    decode_attend<T, D>(list, s_count, q, K, V, dl, partial + ((size_t)bh * nsplit + split) * (D + 2), bh, b, hk, scale_log2, ks_b, ks_l,
                        ks_h, vs_b, vs_l, vs_h);
    if (last_of_row(tickets + bh, nsplit)) combine_row<T, D>(partial, o, lse, nsplit, bh);
}

// ---- incremental decoding: the kept set is carried from step to step --------------------------------------------------
// One key is appended per step, so the set of the w best keys changes by at most one member: the new key enters iff it
// beats the weakest kept key (or the set is not full yet), and that weakest key leaves. The state of a (batch, head) row:
//   int32 [0] count (<= w)   [1] position of the weakest kept key in the list   [2..3] its 64-bit sort key
//         [4..7] unused
//   int32 [8 .. 8 + w)       the kept key indices, in no particular order
// A step costs O(w), whatever the number of cached keys: no scan of the delta row.
constexpr int kStateHeader = 8;
constexpr int kListSplit = 128;            // kept keys per CTA of the list attention kernel (256: 4 us slower per step at w = 2048)

__device__ __forceinline__ int state_stride(int w_cap) { return kStateHeader + ((w_cap + 3) & ~3); }

// what the appended key N - 1 does to a row's set: 0 nothing, 1 appended (set not full), 2 replaces the weakest
__device__ __forceinline__ int step_mode(const int* hdr, int w_cap, unsigned long long kn) {
    const int count = hdr[0];
    if (count < w_cap) return 1;
    const unsigned long long kmin = ((unsigned long long)(unsigned)hdr[3] << 32) | (unsigned)hdr[2];
    return kn > kmin ? 2 : 0;
}

// weakest key of the row's list (entry `skip_pos`, if >= 0, reads as key `skip_j`): written to the header by thread 0
__device__ __forceinline__ void store_weakest(int* hdr, const int* kept, int count, const float* dl, int skip_pos, int skip_j) {
    __shared__ unsigned long long s_key[32];
    __shared__ int s_pos[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = blockDim.x >> 5;
    unsigned long long best = ~0ull;
    int pos = -1;
    for (int i = tid; i < count; i += blockDim.x) {
        const int j = i == skip_pos ? skip_j : kept[i];
        const unsigned long long k = key_of(dl[j], j);
        if (k < best) { best = k; pos = i; }
    }
    for (int o = 16; o; o >>= 1) {
        const unsigned long long k2 = __shfl_xor_sync(0xffffffffu, best, o);
        const int p2 = __shfl_xor_sync(0xffffffffu, pos, o);
        if (k2 < best) { best = k2; pos = p2; }
    }
    if (lane == 0) { s_key[warp] = best; s_pos[warp] = pos; }
    __syncthreads();
    if (tid == 0) {
        for (int wq = 1; wq < nwarp; ++wq)
            if (s_key[wq] < best) { best = s_key[wq]; pos = s_pos[wq]; }
        hdr[1] = pos;
        hdr[2] = (int)(uint32_t)best;
        hdr[3] = (int)(uint32_t)(best >> 32);
    }
}

// after decode_index_kernel has written the kept indices of the first N keys: count and weakest key
__global__ void __launch_bounds__(256) decode_state_init_kernel(const float* __restrict__ delta, int64_t ld, int keep, int w_cap,
                                                                int* __restrict__ state) {
    const int bh = blockIdx.x;
    int* hdr = state + (size_t)bh * state_stride(w_cap);
    if (threadIdx.x == 0) hdr[0] = keep;
    store_weakest(hdr, hdr + kStateHeader, keep, delta + (size_t)bh * ld, -1, 0);
}

// brings a row's state up to date with the appended key N - 1 (every thread of the CTA takes part)
__device__ __forceinline__ void decode_state_update(const float* __restrict__ delta, int64_t ld, int N, int w_cap,
                                                    int* __restrict__ state, int bh) {
    const float* dl = delta + (size_t)bh * ld;
    int* hdr = state + (size_t)bh * state_stride(w_cap);
    int* kept = hdr + kStateHeader;
    const int newj = N - 1, count = hdr[0], weakest = hdr[1];
    const unsigned long long kn = key_of(dl[newj], newj);
    const int mode = step_mode(hdr, w_cap, kn);
    __syncthreads();                                   // every thread has read the header before anyone rewrites it
    if (mode == 0) return;
    if (mode == 1) {                                   // the appended key has the largest index: on equal delta it is the weakest
        if (threadIdx.x == 0) {
            const unsigned long long kmin = ((unsigned long long)(unsigned)hdr[3] << 32) | (unsigned)hdr[2];
            kept[count] = newj;
            hdr[0] = count + 1;
            if (count == 0 || kn < kmin) { hdr[1] = count; hdr[2] = (int)(uint32_t)kn; hdr[3] = (int)(uint32_t)(kn >> 32); }
        }
        return;
    }
    store_weakest(hdr, kept, count, dl, weakest, newj);
    if (threadIdx.x == 0) kept[weakest] = newj;
}

// attention over the row's kept list as it is AFTER the appended key N - 1 is taken into account (the stored state still
// describes the first N - 1 keys; decode_state_update_kernel brings it up to date afterwards)
template <typename T, int D>
__global__ void __launch_bounds__(kAttnThreads) decode_list_attn_kernel(const T* __restrict__ q, const T* __restrict__ K,
                                                                        const T* __restrict__ V, const float* __restrict__ delta,
                                                                        int64_t ld, const int* __restrict__ state, int w_cap,
                                                                        float* __restrict__ partial, int N, int Hq, int G,
                                                                        float scale_log2, int nsplit, int64_t ks_b, int64_t ks_l,
                                                                        int64_t ks_h, int64_t vs_b, int64_t vs_l, int64_t vs_h) {
    __shared__ int list[kListSplit];
    const int split = blockIdx.x, bh = blockIdx.y, b = bh / Hq, h = bh % Hq, hk = h / G;
    const int tid = threadIdx.x;
    const float* dl = delta + (size_t)bh * ld;
    const int* hdr = state + (size_t)bh * state_stride(w_cap);
    const int* kept = hdr + kStateHeader;
    const int newj = N - 1, count = hdr[0];
    const int mode = step_mode(hdr, w_cap, key_of(dl[newj], newj));
    const int eff = count + (mode == 1 ? 1 : 0), weakest = hdr[1];
    const int e = split * kListSplit + tid;
    if (tid < kListSplit && e < eff) list[tid] = (e >= count || (mode == 2 && e == weakest)) ? newj : kept[e];
    __syncthreads();
    decode_attend<T, D>(list, max(0, min(kListSplit, eff - split * kListSplit)), q, K, V, dl,
                        partial + ((size_t)bh * nsplit + split) * (D + 2), bh, b, hk, scale_log2, ks_b, ks_l, ks_h, vs_b, vs_l, vs_h);
}

// The step's second kernel, one CTA of 8 D threads per row: the splits' partials -> o, log-sum-exp, and then, every CTA of
// the attention kernel having read the row's state, the state takes in the appended key. (Doing this in the attention
// kernel's last CTA per row, as dma_decode does, was measured slower here, 16.5 -> 20.7 us per step: the state must then be
// writable in the attention kernel, whose loads of the kept list no longer take the read-only path, and the update, which
// scans the w kept keys, runs on 256 threads at the end of the row's critical path instead of 8 D.)
template <typename T, int D>
__global__ void __launch_bounds__(8 * D) decode_step_combine_kernel(const float* __restrict__ partial, T* __restrict__ o, float* __restrict__ lse,
                                                                    int nsplit, const float* __restrict__ delta, int64_t ld,
                                                                    int N, int w_cap, int* __restrict__ state) {
    __shared__ float s_m[8], s_l[8], s_o[8][D];
    const int bh = blockIdx.x, c = threadIdx.x % D, g = threadIdx.x / D;     // group g takes the splits s = g, g + 8, ...
    const float* p = partial + (size_t)bh * nsplit * (D + 2);
    float mx = -INFINITY;
    for (int s = g; s < nsplit; s += 8) mx = fmaxf(mx, p[(size_t)s * (D + 2) + D]);
    float l = 0.0f, acc = 0.0f;
    for (int s = g; s < nsplit; s += 8) {
        const float ms = p[(size_t)s * (D + 2) + D];
        const float f = ms == -INFINITY ? 0.0f : exp2f(ms - mx);
        l += p[(size_t)s * (D + 2) + D + 1] * f;
        acc += p[(size_t)s * (D + 2) + c] * f;
    }
    s_o[g][c] = acc;
    if (c == 0) { s_m[g] = mx; s_l[g] = l; }
    __syncthreads();
    if (g == 0) {
        float m_all = -INFINITY;
#pragma unroll
        for (int q = 0; q < 8; ++q) m_all = fmaxf(m_all, s_m[q]);
        float lt = 0.0f, at = 0.0f;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float f = s_m[q] == -INFINITY ? 0.0f : exp2f(s_m[q] - m_all);
            lt += s_l[q] * f;
            at += s_o[q][c] * f;
        }
        const float v = lt > 0.0f ? at / lt : 0.0f;
        if constexpr (sizeof(T) == 2) o[(size_t)bh * D + c] = __float2bfloat16_rn(v); else o[(size_t)bh * D + c] = v;
        if (c == 0) lse[bh] = lt > 0.0f ? 0.6931471805599453f * (m_all + log2f(lt)) : -INFINITY;
    }
    // incremental decoding: the attention kernel has read the row's state, which can now take in the appended key
    if (state) decode_state_update(delta, ld, N, w_cap, state, bh);
}



template <typename T, int D>
int launch_typed(const Prob& P, const void* q, const void* K, const void* V, const float* delta, int64_t ld, void* o, float* lse,
                 const unsigned long long* thr, int* tickets, float* partial, int nsplit, cudaStream_t st) {
    decode_attn_kernel<T, D><<<dim3(nsplit, P.B * P.Hq), kAttnThreads, 0, st>>>(
        (const T*)q, (const T*)K, (const T*)V, delta, ld, thr, partial, P.L, P.Hq, P.G, P.scale * 1.4426950408889634f, nsplit, P.ks[0],
        P.ks[1], P.ks[2], P.vs[0], P.vs[1], P.vs[2], tickets, (T*)o, lse);
    count_launch();
    return check_launch();
}

}  // namespace

static int decode_splits(const Prob& P) { return (P.L + kSplitKeys - 1) / kSplitKeys; }

static size_t decode_hist_bytes(const Prob& P) { return (size_t)3 * P.B * P.Hq * 2048 * sizeof(int); }

static int list_splits(const Prob& P) { return (P.w_cap + kListSplit - 1) / kListSplit; }

// header | thresholds | tickets | histograms | partials of the larger of the two attention kernels' split counts
struct DecodeWs {
    unsigned long long* thr;
    int* tickets;
    int* ghist;
    float* partial;
    size_t bytes;
};
static DecodeWs decode_ws(const Prob& P, void* ws) {
    const size_t bh = (size_t)P.B * P.Hq;
    const size_t splits = (size_t)(decode_splits(P) > list_splits(P) ? decode_splits(P) : list_splits(P));
    auto up = [](size_t n) { return (n + 255) / 256 * 256; };
    DecodeWs w;
    size_t off = kWsHeaderBytes;
    char* base = (char*)ws;
    w.thr = reinterpret_cast<unsigned long long*>(base + off); off += up(bh * sizeof(unsigned long long));
    w.tickets = reinterpret_cast<int*>(base + off); off += up(bh * sizeof(int));
    w.ghist = reinterpret_cast<int*>(base + off); off += decode_hist_bytes(P);
    w.partial = reinterpret_cast<float*>(base + off); off += bh * splits * (P.d + 2) * sizeof(float);
    w.bytes = off;
    return w;
}

size_t decode_ws_bytes(const Prob& P) {
    char dummy[1];
    return decode_ws(P, dummy).bytes;
}

size_t decode_state_bytes(const Prob& P) {
    return (size_t)P.B * P.Hq * (kStateHeader + ((P.w_cap + 3) & ~3)) * sizeof(int);
}

// The selection (threshold key per row, tickets zeroed): rows that fit in shared memory are selected by one CTA each in one
// launch; longer rows by the histogram passes spread over CTAs of 8192 keys (a memset and four launches).
static int launch_select(const Prob& P, const float* delta, int64_t ld, const DecodeWs& W, cudaStream_t st) {
    const int BH = P.B * P.Hq, nslices = (P.L + kSliceKeys - 1) / kSliceKeys;
    if (P.L <= kRowSelectMax) {
        const size_t smem = (size_t)P.L * sizeof(uint32_t);
        if (cudaFuncSetAttribute(decode_row_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kRowSelectMax * sizeof(uint32_t))) != cudaSuccess)
            return DMA_ERR_CUDA;
        decode_row_select_kernel<<<(unsigned)BH, kRowSelectThreads, smem, st>>>(delta, ld, P.L, P.w, W.thr, W.tickets);
        count_launch();
        return check_launch();
    }
    // tickets and histograms are adjacent: one memset
    const size_t zero_bytes = (size_t)((char*)W.ghist - (char*)W.tickets) + (P.w < P.L ? decode_hist_bytes(P) : 0);
    if (cudaMemsetAsync(W.tickets, 0, zero_bytes, st) != cudaSuccess) return DMA_ERR_CUDA;
    if (P.w < P.L) {
        const dim3 grid(nslices, (unsigned)BH);
        for (int pass = 0; pass < 3; ++pass)
            decode_hist_kernel<<<grid, 256, 0, st>>>(delta, ld, P.L, P.w, pass, W.ghist, BH);
        count_launch(3);
    }
    decode_thr_kernel<<<(unsigned)BH, 256, 0, st>>>(delta, ld, P.L, P.w, W.ghist, BH, W.thr);
    count_launch();
    return check_launch();
}

int launch_decode(const Prob& P, const void* q, const void* K, const void* V, const float* delta, int64_t ld, void* o, float* lse,
                  int32_t* sel_idx, void* ws, cudaStream_t st) {
    const size_t bh = (size_t)P.B * P.Hq;
    const DecodeWs W = decode_ws(P, ws);
    int rc = launch_select(P, delta, ld, W, st);
    if (rc) return rc;
    if (sel_idx) {
        decode_index_kernel<<<(unsigned)bh, 256, 0, st>>>(delta, ld, P.L, P.w, W.thr, sel_idx, P.w);
        count_launch();
    }
    const int ns = decode_splits(P);
    if (P.dtype == DMA_BF16)
        return P.d == 128 ? launch_typed<__nv_bfloat16, 128>(P, q, K, V, delta, ld, o, lse, W.thr, W.tickets, W.partial, ns, st)
                          : launch_typed<__nv_bfloat16, 64>(P, q, K, V, delta, ld, o, lse, W.thr, W.tickets, W.partial, ns, st);
    return P.d == 128 ? launch_typed<float, 128>(P, q, K, V, delta, ld, o, lse, W.thr, W.tickets, W.partial, ns, st)
                      : launch_typed<float, 64>(P, q, K, V, delta, ld, o, lse, W.thr, W.tickets, W.partial, ns, st);
}

// Builds the incremental state from the first N = P.L cached keys: the selection, the kept indices into the state's
// lists, then count and weakest key.
int launch_decode_state_init(const Prob& P, const float* delta, int64_t ld, int* state, void* ws, cudaStream_t st) {
    const size_t bh = (size_t)P.B * P.Hq;
    const DecodeWs W = decode_ws(P, ws);
    int rc = launch_select(P, delta, ld, W, st);
    if (rc) return rc;
    const int stride = kStateHeader + ((P.w_cap + 3) & ~3);
    decode_index_kernel<<<(unsigned)bh, 256, 0, st>>>(delta, ld, P.L, P.w, W.thr, state + kStateHeader, stride);
    decode_state_init_kernel<<<(unsigned)bh, 256, 0, st>>>(delta, ld, P.w, P.w_cap, state);
    count_launch(2);
    return check_launch();
}

template <typename T, int D>
static int launch_step_typed(const Prob& P, const void* q, const void* K, const void* V, const float* delta, int64_t ld, int* state,
                             void* o, float* lse, float* partial, cudaStream_t st) {
    const int ns = list_splits(P);
    decode_list_attn_kernel<T, D><<<dim3(ns, P.B * P.Hq), kAttnThreads, 0, st>>>(
        (const T*)q, (const T*)K, (const T*)V, delta, ld, state, P.w_cap, partial, P.L, P.Hq, P.G, P.scale * 1.4426950408889634f, ns,
        P.ks[0], P.ks[1], P.ks[2], P.vs[0], P.vs[1], P.vs[2]);
    decode_step_combine_kernel<T, D><<<P.B * P.Hq, 8 * D, 0, st>>>(partial, (T*)o, lse, ns, delta, ld, P.L, P.w_cap, state);
    count_launch(2);
    return check_launch();
}

// One decoding step with the carried state: P.L counts the cached keys INCLUDING the one appended for this step.
int launch_decode_step(const Prob& P, const void* q, const void* K, const void* V, const float* delta, int64_t ld, int* state,
                       void* o, float* lse, void* ws, cudaStream_t st) {
    float* partial = decode_ws(P, ws).partial;
    if (P.dtype == DMA_BF16)
        return P.d == 128 ? launch_step_typed<__nv_bfloat16, 128>(P, q, K, V, delta, ld, state, o, lse, partial, st)
                          : launch_step_typed<__nv_bfloat16, 64>(P, q, K, V, delta, ld, state, o, lse, partial, st);
    return P.d == 128 ? launch_step_typed<float, 128>(P, q, K, V, delta, ld, state, o, lse, partial, st)
                      : launch_step_typed<float, 64>(P, q, K, V, delta, ld, state, o, lse, partial, st);
}

}  // namespace dma
