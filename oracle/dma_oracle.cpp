// CPU oracle for Dynamic Mask Attention (DMA).
//
// TEST INFRASTRUCTURE ONLY. This file is the plain, slow, obviously-correct statement of what the
// hot path computes. It is used by the tests, by the smoke check and by the benchmark's CPU-baseline
// leg, never by the product path, and it shares no code, header, table or helper with the CUDA
// kernels. Every routine follows the definition (or the algorithm's steps) in the paper's order:
// no tiling, no fusion, no SIMD intrinsics; OpenMP only spreads independent rows / keys over cores.
//
//   delta            Eq. (delta_calc) of Sec. 4.1 and the listing of App. A: dt = exp(A * softplus(v . W)), with
//                    W per head over the head's own d channels, or (delta_full) over all Hkv*d channels of the row
//   selection        Eq. (mask_combine) of Sec. 4.1 read per query row as the App. A listing does
//                    (top-w over the causally visible keys), ties broken toward the lower index
//   block bitmap     the Judge(M_j) block test of Alg. 1 / Alg. 2, per (query tile, key tile)
//   forward          Eq. (attention_output) of Sec. 4.2 / Eq. (forward_pass) of Sec. 4.3
//   backward         Eqs. (grad_v), (grad_s), (grad_m), (grad_qk) of Sec. 4.3, summed over query steps
//                    as Alg. 2 does; dM is the column sum of dS over query rows
//
// Parity status: every routine is pinned by the CPU test-suite to closed forms, invariants, brute
// force or textbook special cases, with ONE exception: the *bit pattern* of delta. The paper fixes
// no precision or operation order for delta, so the order used here ("delta-v1", documented below)
// is this build's own specification: delta's bits are "parity unpinned" by the paper; its value is
// pinned to an fp64 evaluation of the formula within a few ulp.
//
// Layouts (all contiguous, row-major):  Q,O,dO,dQ [B,L,Hq,d]   K,V,dK,dV [B,L,Hkv,d]
//                                       delta/bias, expiry, lse, dM [B,Hq,L]   keep [B,Hq,L,L] (tiny cases)
// Query head h reads KV head h / (Hq/Hkv).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <queue>
#include <vector>

namespace {

// ----------------------------------------------------------------------------------------------
// delta-v1: a fixed sequence of correctly-rounded IEEE fp32 operations (compiled with
// -ffp-contract=off, no fast-math), so that any IEEE machine produces the same bits.
// ----------------------------------------------------------------------------------------------

// exp(x) for x clamped to [-87, 88]: n = rint(x*log2(e)) by the 1.5*2^23 trick, two-constant
// Cody-Waite reduction, degree-7 Taylor polynomial by Horner (one fma per step), exact scaling by 2^n.
float exp_spec(float x) {
    x = std::fmin(std::fmax(x, -87.0f), 88.0f);
    const float magic = 12582912.0f;                       // 1.5 * 2^23
    float t = x * 0x1.715476p+0f;                          // x * log2(e), rounded once
    float n = (t + magic) - magic;                         // nearest integer, ties to even
    float r = std::fmaf(n, -0x1.62e4p-1f, x);              // exact: ln2_hi has 15 significant bits
    r = std::fmaf(n, -0x1.7f7d1cp-20f, r);
    float q = 0x1.a01a02p-13f;                             // 1/7!
    q = std::fmaf(q, r, 0x1.6c16c2p-10f);                  // 1/6!
    q = std::fmaf(q, r, 0x1.111112p-7f);                   // 1/5!
    q = std::fmaf(q, r, 0x1.555556p-5f);                   // 1/4!
    q = std::fmaf(q, r, 0x1.555556p-3f);                   // 1/3!
    q = std::fmaf(q, r, 0.5f);
    q = std::fmaf(q, r, 1.0f);
    q = std::fmaf(q, r, 1.0f);
    int32_t e = (int32_t)n;                                // in [-126, 127]
    uint32_t bits = (uint32_t)(e + 127) << 23;             // the float 2^e
    float two_n;
    std::memcpy(&two_n, &bits, 4);
    return q * two_n;
}

// log(1+t) for 0 < t <= 1 as 2*atanh(s), s = t/(2+t): 8-term odd series by Horner in s^2.
float log1p_spec(float t) {
    float s = t / (2.0f + t);
    float u = s * s;
    float q = 0x1.111112p-4f;                              // 1/15
    q = std::fmaf(q, u, 0x1.3b13b2p-4f);                   // 1/13
    q = std::fmaf(q, u, 0x1.745d18p-4f);                   // 1/11
    q = std::fmaf(q, u, 0x1.c71c72p-4f);                   // 1/9
    q = std::fmaf(q, u, 0x1.24924ap-3f);                   // 1/7
    q = std::fmaf(q, u, 0x1.99999ap-3f);                   // 1/5
    q = std::fmaf(q, u, 0x1.555556p-2f);                   // 1/3
    q = std::fmaf(q, u, 1.0f);
    return (2.0f * s) * q;
}

float softplus_spec(float z) {
    return std::fmax(z, 0.0f) + log1p_spec(exp_spec(-std::fabs(z)));
}

// z = v . W: eight-channel partial sums (left-to-right fma chains from 0) combined by a balanced
// pairwise tree of adjacent partials. d must be 8 * (power of two).
float dot_spec(const float* v, const float* w, int d) {
    float part[64];
    int n = d / 8;
    for (int k = 0; k < n; ++k) {
        float p = 0.0f;
        for (int c = 8 * k; c < 8 * k + 8; ++c) p = std::fmaf(v[c], w[c], p);
        part[k] = p;
    }
    while (n > 1) {
        for (int k = 0; k < n / 2; ++k) part[k] = part[2 * k] + part[2 * k + 1];
        n /= 2;
    }
    return part[0];
}

// Strict total order used everywhere a key "beats" another: larger delta first, then lower index.
inline bool beats(float da, int ia, float db, int ib) {
    return da > db || (da == db && ia < ib);
}

// ----------------------------------------------------------------------------------------------
// attention rows
// ----------------------------------------------------------------------------------------------

template <class T>
struct Problem {
    int B, L, Hq, Hkv, d;
    T scale;
    const T *Q, *K, *V, *bias;
    const int32_t* expiry;   // [B,Hq,L] or null
    const uint8_t* keep;     // [B,Hq,L,L] or null (definition form; tiny cases)
    int causal;              // 1: row i sees keys j <= i (the listing's causal fill); 0: every row sees every key
                             // (the listing with an all-zero causal_m), key j kept by the rows i < expiry[j]
    int jlast(int i) const { return causal ? i : L - 1; }    // last key row i can see
    int ifirst(int j) const { return causal ? j : 0; }       // first row that can see key j
    int G() const { return Hq / Hkv; }
    const T* q(int b, int i, int h) const { return Q + (((size_t)b * L + i) * Hq + h) * d; }
    const T* k(int b, int j, int hk) const { return K + (((size_t)b * L + j) * Hkv + hk) * d; }
    const T* v(int b, int j, int hk) const { return V + (((size_t)b * L + j) * Hkv + hk) * d; }
    bool kept(int b, int h, int i, int j) const {
        if (causal && j > i) return false;
        size_t bh = (size_t)b * Hq + h;
        if (keep) return keep[(bh * L + i) * L + j] != 0;
        return expiry[bh * L + j] > i;
    }
};

// One query row of Eq. (forward_pass): scores over the kept set, softmax, weighted value sum.
// Returns the kept indices and their probabilities; o (d values) and lse are written if non-null.
template <class T>
void row_forward(const Problem<T>& P, int b, int h, int i, std::vector<int>& idx, std::vector<T>& p,
                 T* o, T* lse) {
    const int hk = h / P.G();
    const T* qi = P.q(b, i, h);
    const T* bias = P.bias + ((size_t)b * P.Hq + h) * P.L;
    idx.clear();
    p.clear();
    for (int j = 0; j <= P.jlast(i); ++j)
        if (P.kept(b, h, i, j)) idx.push_back(j);
    T m = -INFINITY;
    for (int j : idx) {
        const T* kj = P.k(b, j, hk);
        T s = 0;
        for (int c = 0; c < P.d; ++c) s += qi[c] * kj[c];
        s = s * P.scale + bias[j];
        p.push_back(s);
        m = std::max(m, s);
    }
    T sum = 0;
    for (T& s : p) {
        s = std::exp(s - m);
        sum += s;
    }
    for (T& s : p) s /= sum;
    if (lse) *lse = m + std::log(sum);
    if (o) {
        for (int c = 0; c < P.d; ++c) o[c] = 0;
        for (size_t t = 0; t < idx.size(); ++t) {
            const T* vj = P.v(b, idx[t], hk);
            for (int c = 0; c < P.d; ++c) o[c] += p[t] * vj[c];
        }
    }
}

template <class T>
int forward(const Problem<T>& P, const int32_t* rows, int nrows, T* O, T* LSE) {
    // rows == null: every row, outputs [B,L,Hq,d] / [B,Hq,L]; else only the listed rows,
    // outputs compact [B,nrows,Hq,d] / [B,Hq,nrows].
    const int R = rows ? nrows : P.L;
    const long total = (long)P.B * P.Hq * R;
#pragma omp parallel
    {
        std::vector<int> idx;
        std::vector<T> p;
#pragma omp for schedule(dynamic, 16)
        for (long t = 0; t < total; ++t) {
            int r = (int)(t % R);
            int h = (int)((t / R) % P.Hq);
            int b = (int)(t / ((long)R * P.Hq));
            int i = rows ? rows[r] : r;
            T lse;
            row_forward(P, b, h, i, idx, p, O + (((size_t)b * R + r) * P.Hq + h) * P.d, &lse);
            LSE[((size_t)b * P.Hq + h) * R + r] = lse;
        }
    }
    return 0;
}

// Backward of Sec. 4.3. Pass 1 (per query row): forward quantities, D_i = dO_i . o_i, and dQ_i. Alg. 2 takes O
// as an input read back from memory (D_i = rowsum(dO_i o O_i)), so when Ostored is given (the forward output as
// it was stored, i.e. rounded to the element type) D uses it; when it is null D uses the exact o of this pass.
// Pass 2 (per key): dV_j, dK_j (summed over the query heads sharing the KV head) and dM_j, each a
// sum over the query rows that keep key j. keys == null: all keys; else only the listed keys, with
// compact outputs dK,dV [B,nkeys,Hkv,d], dM [B,Hq,nkeys]; dQ may be null to skip it.
template <class T>
int backward(const Problem<T>& P, const T* Ostored, const T* dO, const int32_t* keys, int nkeys, T* dQ, T* dK,
             T* dV, T* dM) {
    const int L = P.L, d = P.d, Hq = P.Hq, Hkv = P.Hkv, G = P.G();
    std::vector<T> LSE((size_t)P.B * Hq * L), D((size_t)P.B * Hq * L);
    std::vector<uint8_t> need((size_t)P.B * Hq * L, keys ? 0 : 1);
    if (keys) {
        // only rows that keep one of the listed keys are needed for pass 2
        for (int b = 0; b < P.B; ++b)
            for (int h = 0; h < Hq; ++h)
                for (int t = 0; t < nkeys; ++t)
                    for (int i = P.ifirst(keys[t]); i < L; ++i)
                        if (P.kept(b, h, i, keys[t])) need[((size_t)b * Hq + h) * L + i] = 1;
        if (dQ) std::fill(need.begin(), need.end(), 1);
    }
    const long total = (long)P.B * Hq * L;
#pragma omp parallel
    {
        std::vector<int> idx;
        std::vector<T> p, o(d);
#pragma omp for schedule(dynamic, 16)
        for (long t = 0; t < total; ++t) {
            int i = (int)(t % L);
            int h = (int)((t / L) % Hq);
            int b = (int)(t / ((long)L * Hq));
            size_t bhi = ((size_t)b * Hq + h) * L + i;
            if (!need[bhi]) continue;
            const int hk = h / G;
            T lse;
            row_forward(P, b, h, i, idx, p, o.data(), &lse);
            const T* doi = dO + (((size_t)b * L + i) * Hq + h) * d;
            const T* oi = Ostored ? Ostored + (((size_t)b * L + i) * Hq + h) * d : o.data();
            T Di = 0;
            for (int c = 0; c < d; ++c) Di += doi[c] * oi[c];
            LSE[bhi] = lse;
            D[bhi] = Di;
            if (dQ) {
                T* dqi = dQ + (((size_t)b * L + i) * Hq + h) * d;
                for (int c = 0; c < d; ++c) dqi[c] = 0;
                for (size_t u = 0; u < idx.size(); ++u) {
                    const T* vj = P.v(b, idx[u], hk);
                    const T* kj = P.k(b, idx[u], hk);
                    T dp = 0;
                    for (int c = 0; c < d; ++c) dp += doi[c] * vj[c];
                    T ds = p[u] * (dp - Di);
                    for (int c = 0; c < d; ++c) dqi[c] += ds * kj[c] * P.scale;
                }
            }
        }
    }
    const int NK = keys ? nkeys : L;
    const long totalk = (long)P.B * Hkv * NK;
#pragma omp parallel for schedule(dynamic, 4)
    for (long t = 0; t < totalk; ++t) {
        int r = (int)(t % NK);
        int hk = (int)((t / NK) % Hkv);
        int b = (int)(t / ((long)NK * Hkv));
        int j = keys ? keys[r] : r;
        T* dkj = dK + (((size_t)b * NK + r) * Hkv + hk) * d;
        T* dvj = dV + (((size_t)b * NK + r) * Hkv + hk) * d;
        for (int c = 0; c < d; ++c) dkj[c] = dvj[c] = 0;
        const T* kj = P.k(b, j, hk);
        const T* vj = P.v(b, j, hk);
        for (int h = hk * G; h < (hk + 1) * G; ++h) {
            size_t bh = (size_t)b * Hq + h;
            T dm = 0;
            for (int i = P.ifirst(j); i < L; ++i) {
                if (!P.kept(b, h, i, j)) continue;
                const T* qi = P.q(b, i, h);
                const T* doi = dO + (((size_t)b * L + i) * Hq + h) * d;
                T s = 0, dp = 0;
                for (int c = 0; c < d; ++c) s += qi[c] * kj[c];
                s = s * P.scale + P.bias[bh * L + j];
                T p = std::exp(s - LSE[bh * L + i]);
                for (int c = 0; c < d; ++c) dp += doi[c] * vj[c];
                T ds = p * (dp - D[bh * L + i]);
                for (int c = 0; c < d; ++c) {
                    dvj[c] += p * doi[c];
                    dkj[c] += ds * qi[c] * P.scale;
                }
                dm += ds;
            }
            dM[bh * NK + r] = dm;
        }
    }
    return 0;
}

// dQ of Sec. 4.3 (Eq. grad_qk, first line) on a subset of query rows. dQ_i depends on row i alone:
// dQ_i = scale * sum_{j in I_i} dS_ij k_j with dS_ij = p_ij (dO_i . v_j - D_i), D_i = dO_i . O_i (Alg. 2 reads
// the stored O: Ostored holds it for the listed rows, compact [B,nrows,Hq,d]; null = the exact o of this row).
// The same statements as pass 1 of `backward`, restricted to the listed rows; output compact [B,nrows,Hq,d].
template <class T>
int backward_dq_rows(const Problem<T>& P, const T* Ostored, const T* dO, const int32_t* rows, int nrows, T* dQ) {
    const int L = P.L, d = P.d, Hq = P.Hq, G = P.G();
    const long total = (long)P.B * Hq * nrows;
#pragma omp parallel
    {
        std::vector<int> idx;
        std::vector<T> p, o(d);
#pragma omp for schedule(dynamic, 1)
        for (long t = 0; t < total; ++t) {
            int r = (int)(t % nrows);
            int h = (int)((t / nrows) % Hq);
            int b = (int)(t / ((long)nrows * Hq));
            const int i = rows[r], hk = h / G;
            row_forward(P, b, h, i, idx, p, o.data(), (T*)nullptr);
            const T* doi = dO + (((size_t)b * L + i) * Hq + h) * d;
            const T* oi = Ostored ? Ostored + (((size_t)b * nrows + r) * Hq + h) * d : o.data();
            T Di = 0;
            for (int c = 0; c < d; ++c) Di += doi[c] * oi[c];
            T* dqi = dQ + (((size_t)b * nrows + r) * Hq + h) * d;
            for (int c = 0; c < d; ++c) dqi[c] = 0;
            for (size_t u = 0; u < idx.size(); ++u) {
                const T* vj = P.v(b, idx[u], hk);
                const T* kj = P.k(b, idx[u], hk);
                T dp = 0;
                for (int c = 0; c < d; ++c) dp += doi[c] * vj[c];
                T ds = p[u] * (dp - Di);
                for (int c = 0; c < d; ++c) dqi[c] += ds * kj[c] * P.scale;
            }
        }
    }
    return 0;
}

template <class T>
Problem<T> make_problem(int B, int L, int Hq, int Hkv, int d, double scale, const T* Q, const T* K,
                        const T* V, const T* bias, const int32_t* expiry, const uint8_t* keep, int causal) {
    Problem<T> P;
    P.causal = causal;
    P.B = B; P.L = L; P.Hq = Hq; P.Hkv = Hkv; P.d = d;
    P.scale = (T)scale;
    P.Q = Q; P.K = K; P.V = V; P.bias = bias; P.expiry = expiry; P.keep = keep;
    return P;
}

}  // namespace

extern "C" {

// Single-value access to the delta-v1 scalar routines (used by the pin tests).
float dmao_exp_spec(float x) { return exp_spec(x); }
float dmao_log1p_spec(float t) { return log1p_spec(t); }
float dmao_softplus_spec(float z) { return softplus_spec(z); }

// Sec. 4.1, Eq. (delta_calc): z[b,h,j] = V[b,j,h/G,:] . W[h,:];  delta = exp(A[h] * softplus(z)).
int dmao_delta(const float* V, const float* W, const float* A, int B, int L, int Hq, int Hkv, int d,
               float* z_out, float* delta) {
    if (d % 8 || (d / 8) & (d / 8 - 1) || d > 512 || Hq % Hkv) return -1;
    const int G = Hq / Hkv;
#pragma omp parallel for collapse(2)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < Hq; ++h)
            for (int j = 0; j < L; ++j) {
                const float* v = V + (((size_t)b * L + j) * Hkv + h / G) * d;
                float z = dot_spec(v, W + (size_t)h * d, d);
                float sp = softplus_spec(z);
                size_t o = ((size_t)b * Hq + h) * L + j;
                if (z_out) z_out[o] = z;
                delta[o] = exp_spec(A[h] * sp);
            }
    return 0;
}

// Eq. (delta_calc) with the sampling weights as the paper states them, a map from all heads' value channels to
// one score per head (App. A listing: a linear layer over the value row flattened to Hkv*d channels):
//   z[b,h,j] = sum_{h'} V[b,j,h',:] . W[h, h'*d : (h'+1)*d]
// delta-v1 order: the per-head dot products as above, added over h' = 0, 1, ... from left to right (one rounded
// addition each, starting from the h' = 0 term).
int dmao_delta_full(const float* V, const float* W, const float* A, int B, int L, int Hq, int Hkv, int d,
                    float* z_out, float* delta) {
    if (d % 8 || (d / 8) & (d / 8 - 1) || d > 512) return -1;
#pragma omp parallel for collapse(2)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < Hq; ++h)
            for (int j = 0; j < L; ++j) {
                const float* v = V + ((size_t)b * L + j) * Hkv * d;
                const float* w = W + (size_t)h * Hkv * d;
                float z = dot_spec(v, w, d);
                for (int hk = 1; hk < Hkv; ++hk) z = z + dot_spec(v + (size_t)hk * d, w + (size_t)hk * d, d);
                float sp = softplus_spec(z);
                size_t o = ((size_t)b * Hq + h) * L + j;
                if (z_out) z_out[o] = z;
                delta[o] = exp_spec(A[h] * sp);
            }
    return 0;
}

// Selection, definition form (App. A listing: causal fill, then top-k per query row): for row i the
// visible keys 0..i are ordered by (delta descending, index ascending) and the first min(w, i+1)
// are kept. keep is [BH, L, L] with 1 = kept.
int dmao_select_definition(const float* delta, int BH, int L, int w, uint8_t* keep) {
#pragma omp parallel for collapse(2) schedule(dynamic, 8)
    for (int bh = 0; bh < BH; ++bh)
        for (int i = 0; i < L; ++i) {
            const float* dl = delta + (size_t)bh * L;
            uint8_t* row = keep + ((size_t)bh * L + i) * L;
            std::memset(row, 0, L);
            std::vector<int> order(i + 1);
            for (int j = 0; j <= i; ++j) order[j] = j;
            std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return dl[a] > dl[b]; });
            int n = std::min(w, i + 1);
            for (int t = 0; t < n; ++t) row[order[t]] = 1;
        }
    return 0;
}

// Selection, interval form. Under the strict order `beats`, the number of visible keys beating key j
// only grows with the row index, so j is kept exactly for rows j <= i < expiry[j]. Sequential
// algorithm: walk the rows; hold the current kept set in a heap whose top is the worst key; when the
// set exceeds w, the worst key x leaves for good at this row: expiry[x] = i. Survivors get L.
int dmao_select_expiry(const float* delta, int BH, int L, int w, int32_t* expiry) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < BH; ++bh) {
        const float* dl = delta + (size_t)bh * L;
        int32_t* e = expiry + (size_t)bh * L;
        auto worse_on_top = [&](int a, int b) { return beats(dl[a], a, dl[b], b); };
        std::priority_queue<int, std::vector<int>, decltype(worse_on_top)> heap(worse_on_top);
        for (int i = 0; i < L; ++i) {
            heap.push(i);
            if ((int)heap.size() > w) {
                e[heap.top()] = i;
                heap.pop();
            }
        }
        while (!heap.empty()) {
            e[heap.top()] = L;
            heap.pop();
        }
    }
    return 0;
}

int dmao_keep_from_expiry(const int32_t* expiry, int BH, int L, uint8_t* keep) {
    for (int bh = 0; bh < BH; ++bh)
        for (int i = 0; i < L; ++i)
            for (int j = 0; j < L; ++j)
                keep[((size_t)bh * L + i) * L + j] = (j <= i && expiry[(size_t)bh * L + j] > i) ? 1 : 0;
    return 0;
}

// Block activity (the Judge test of Alg. 1 / Alg. 2 per (query tile, key tile)): bit kt of row qt is
// set iff some (i, j) in the tile is kept. bitmap is [BH, Tr, ceil(Tc/32)] uint32.
int dmao_bitmap_definition(const uint8_t* keep, int BH, int L, int bm, int bn, uint32_t* bitmap) {
    const int Tr = (L + bm - 1) / bm, Tc = (L + bn - 1) / bn, Wd = (Tc + 31) / 32;
    std::memset(bitmap, 0, (size_t)BH * Tr * Wd * 4);
    for (int bh = 0; bh < BH; ++bh)
        for (int i = 0; i < L; ++i)
            for (int j = 0; j < L; ++j)
                if (keep[((size_t)bh * L + i) * L + j])
                    bitmap[((size_t)bh * Tr + i / bm) * Wd + (j / bn) / 32] |= 1u << ((j / bn) % 32);
    return 0;
}

// Non-causal mode: key j is kept by the rows 0 <= i < expiry[j] (expiry is L for the w selected keys, 0 otherwise).
int dmao_keep_from_expiry_noncausal(const int32_t* expiry, int BH, int L, uint8_t* keep) {
    for (int bh = 0; bh < BH; ++bh)
        for (int i = 0; i < L; ++i)
            for (int j = 0; j < L; ++j) keep[((size_t)bh * L + i) * L + j] = expiry[(size_t)bh * L + j] > i ? 1 : 0;
    return 0;
}

int dmao_bitmap_from_expiry(const int32_t* expiry, int BH, int L, int bm, int bn, uint32_t* bitmap) {
    const int Tr = (L + bm - 1) / bm, Tc = (L + bn - 1) / bn, Wd = (Tc + 31) / 32;
    std::memset(bitmap, 0, (size_t)BH * Tr * Wd * 4);
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < BH; ++bh)
        for (int qt = 0; qt < Tr; ++qt) {
            const int qs = qt * bm, qe = std::min(L, qs + bm) - 1;
            for (int j = 0; j <= qe; ++j) {
                // key j is kept by some row of [qs, qe] iff the rows [max(qs,j), qe] meet [j, expiry)
                if (expiry[(size_t)bh * L + j] > std::max(qs, j))
                    bitmap[((size_t)bh * Tr + qt) * Wd + (j / bn) / 32] |= 1u << ((j / bn) % 32);
            }
        }
    return 0;
}

#define DMAO_FWD(NAME, T)                                                                            \
    int NAME(const T* Q, const T* K, const T* V, const T* bias, const int32_t* expiry,               \
             const uint8_t* keep, int B, int L, int Hq, int Hkv, int d, double scale,                \
             const int32_t* rows, int nrows, T* O, T* LSE, int causal) {                             \
        if (Hq % Hkv || (!expiry && !keep)) return -1;                                               \
        return forward<T>(make_problem<T>(B, L, Hq, Hkv, d, scale, Q, K, V, bias, expiry, keep, causal), \
                          rows, nrows, O, LSE);                                                      \
    }
DMAO_FWD(dmao_fwd_f32, float)
DMAO_FWD(dmao_fwd_f64, double)

#define DMAO_BWD(NAME, T)                                                                            \
    int NAME(const T* Q, const T* K, const T* V, const T* Ostored, const T* dO, const T* bias,       \
             const int32_t* expiry, const uint8_t* keep, int B, int L, int Hq, int Hkv, int d, double scale, \
             const int32_t* keys, int nkeys, T* dQ, T* dK, T* dV, T* dM, int causal) {               \
        if (Hq % Hkv || (!expiry && !keep)) return -1;                                               \
        return backward<T>(make_problem<T>(B, L, Hq, Hkv, d, scale, Q, K, V, bias, expiry, keep, causal), \
                           Ostored, dO, keys, nkeys, dQ, dK, dV, dM);                                         \
    }
DMAO_BWD(dmao_bwd_f32, float)
DMAO_BWD(dmao_bwd_f64, double)

#define DMAO_DQ_ROWS(NAME, T)                                                                        \
    int NAME(const T* Q, const T* K, const T* V, const T* Ostored, const T* dO, const T* bias,       \
             const int32_t* expiry, const uint8_t* keep, int B, int L, int Hq, int Hkv, int d, double scale, \
             const int32_t* rows, int nrows, T* dQ, int causal) {                                    \
        if (Hq % Hkv || (!expiry && !keep) || !rows) return -1;                                      \
        return backward_dq_rows<T>(make_problem<T>(B, L, Hq, Hkv, d, scale, Q, K, V, bias, expiry, keep, causal), \
                                   Ostored, dO, rows, nrows, dQ);                                    \
    }
DMAO_DQ_ROWS(dmao_dq_rows_f32, float)
DMAO_DQ_ROWS(dmao_dq_rows_f64, double)

}  // extern "C"
