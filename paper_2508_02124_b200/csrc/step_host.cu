// dma_step_host: the whole hot path (mask build, forward, optional backward) on HOST buffers, for callers that
// keep their tensors in host memory and for end-to-end timing. Inputs are copied to a caller-provided device
// arena (on helper streams, overlapped with the kernels), the three stages run on the caller's stream, results are
// copied back, and the stream is synchronised.
//
// Every (batch entry, group of KV heads) is an independent problem (the mask is per head, dK and dV are summed only
// inside a KV head's group of query heads), so the step is cut into such groups and pipelined: while group g runs its
// kernels, group g + 1's inputs arrive and group g - 1's results leave. A group is addressed inside the full tensors
// by pointer offsets and the full tensors' strides (the kernels take strides), its copies are strided 2-D copies.
#include "common.cuh"

namespace dma {
namespace {

constexpr int kMaxGroups = 64;

struct Arena {
    size_t off = 0;
    size_t take(size_t bytes) {
        size_t o = off;
        off += (bytes + 255) / 256 * 256;
        return o;
    }
};

struct Layout {
    size_t Q, K, V, dO, O, dQ, dK, dV, W, A, bias, expiry, bitmap, lse, dM, ws_mask, ws_fwd, ws_bwd, total;
    size_t nq, nk, nbh, nbmp, m_ws, f_ws, b_ws, esz, wbytes;
    int head_groups;       // groups of KV heads per batch entry (1 = whole batch entries)
    int groups;            // B * head_groups (1: the whole problem at once)
    int group_batch;       // batch entries per group: 1, or B when there is a single group
    size_t gh, gbmp;       // entries of a group's block of bias / expiry / lse / dM and of its bitmap, padded to 256 bytes
};

// Head groups per batch entry: up to 4, a divisor of Hkv, and only where every per-group pointer stays 16-byte aligned,
// the group is independent (the full sampling weights read all KV heads) and a group's K / V rows are at least 512 bytes wide (measured at L = 16384, 32 / 8 heads: 4 groups of
// 512-byte rows 10.2 ms per step, 8 groups of 256-byte rows 14.6 ms, one group 14.8 ms: short rows slow the copies down).
int pick_head_groups(const Prob& P) {
    if (P.flags & DMA_FLAG_FULL_DELTA) return 1;
    const size_t esz = P.dtype == DMA_BF16 ? 2 : 4;
    for (int g = 4; g > 1; --g) {
        if (P.Hkv % g || (size_t)(P.Hkv / g) * P.d * esz < 512) continue;
        const size_t hq = (size_t)P.Hq / g;
        if (hq % 4) continue;                       // W_delta and A of a group start at its first query head
        return g;
    }
    return 1;
}

int make_layout(const dma_problem_t* p, int backward, Layout* Lo) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    for (int i = 0; i < 3; ++i)
        if (p->q_stride[i] || p->k_stride[i] || p->v_stride[i] || p->o_stride[i]) return DMA_ERR_UNSUPPORTED;
    if ((rc = dma_query_workspace(p, &Lo->m_ws, &Lo->f_ws, &Lo->b_ws))) return rc;
    Lo->head_groups = pick_head_groups(P);
    if ((size_t)P.B * Lo->head_groups > (size_t)kMaxGroups) Lo->head_groups = 1;
    Lo->groups = P.B <= kMaxGroups ? P.B * Lo->head_groups : 1;
    if (Lo->groups == 1) Lo->head_groups = 1;
    // one status header per group in front of each workspace (a group's header is never inside a later group's data)
    Lo->f_ws += (size_t)Lo->groups * kWsHeaderBytes;
    Lo->b_ws += (size_t)Lo->groups * kWsHeaderBytes;
    Lo->esz = P.dtype == DMA_BF16 ? 2 : 4;
    Lo->nq = (size_t)P.B * P.L * P.Hq * P.d;
    Lo->nk = (size_t)P.B * P.L * P.Hkv * P.d;
    Lo->nbh = (size_t)P.B * P.Hq * P.L;
    Lo->nbmp = (size_t)P.B * P.Hq * P.Tr * P.Wd;
    Arena a;
    Lo->Q = a.take(Lo->nq * Lo->esz); Lo->K = a.take(Lo->nk * Lo->esz); Lo->V = a.take(Lo->nk * Lo->esz);
    Lo->O = a.take(Lo->nq * Lo->esz);
    Lo->wbytes = (size_t)P.Hq * ((P.flags & DMA_FLAG_FULL_DELTA) ? P.Hkv * P.d : P.d) * 4;
    Lo->W = a.take(Lo->wbytes); Lo->A = a.take((size_t)P.Hq * 4);
    // per-head vectors and the bitmap live in one padded block per group, so that every group's pointers are aligned
    // whatever Hq * L is
    Lo->group_batch = Lo->groups == 1 ? P.B : 1;
    const size_t hq_g = (size_t)Lo->group_batch * (P.Hq / Lo->head_groups);
    Lo->gh = (hq_g * P.L + 63) / 64 * 64;
    Lo->gbmp = (hq_g * P.Tr * P.Wd + 63) / 64 * 64;
    const size_t vec = (size_t)Lo->groups * Lo->gh * 4;
    Lo->bias = a.take(vec); Lo->expiry = a.take(vec); Lo->bitmap = a.take((size_t)Lo->groups * Lo->gbmp * 4);
    Lo->lse = a.take(vec);
    Lo->ws_mask = a.take(Lo->m_ws); Lo->ws_fwd = a.take(Lo->f_ws);
    if (backward) {
        Lo->dO = a.take(Lo->nq * Lo->esz); Lo->dQ = a.take(Lo->nq * Lo->esz);
        Lo->dK = a.take(Lo->nk * Lo->esz); Lo->dV = a.take(Lo->nk * Lo->esz);
        Lo->dM = a.take(vec); Lo->ws_bwd = a.take(Lo->b_ws);
    }
    Lo->total = a.off;
    return DMA_OK;
}

}  // namespace
}  // namespace dma

using namespace dma;

extern "C" {

int dma_step_host_arena(const dma_problem_t* p, int backward, size_t* bytes) {
    Layout Lo;
    int rc = make_layout(p, backward, &Lo);
    if (rc) return rc;
    if (!bytes) return DMA_ERR_NULL;
    *bytes = Lo.total;
    return DMA_OK;
}

int dma_step_host(const dma_problem_t* p, int backward, const void* hQ, const void* hK, const void* hV, const void* hdO,
                  const float* hW_delta, const float* hA, void* hO, float* hlse, void* hdQ, void* hdK, void* hdV,
                  float* hdM, void* dev_arena, size_t arena_bytes, void* cuda_stream) {
    Layout Lo;
    int rc = make_layout(p, backward, &Lo);
    if (rc) return rc;
    if (!hQ || !hK || !hV || !hW_delta || !hA || !hO || !hlse) return DMA_ERR_NULL;
    if (backward && (!hdO || !hdQ || !hdK || !hdV || !hdM)) return DMA_ERR_NULL;
    if (!dev_arena || arena_bytes < Lo.total || (reinterpret_cast<uintptr_t>(dev_arena) & 255)) return DMA_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    char* a = (char*)dev_arena;
    const int NG = Lo.groups, HG = Lo.head_groups;
    const int L = p->L, d = p->d, nqh = p->Hq / HG, nkh = p->Hkv / HG;
    const int GB = Lo.group_batch;                 // batch entries per group
    const size_t rows = (size_t)GB * L;            // sequence rows per group (batch entries are contiguous)
    const size_t hl = (size_t)GB * nqh * L;        // entries of a group's per-head vectors
    const size_t esz = Lo.esz;

    // Copies run on two helper streams of this call (created and destroyed here: no state is kept) so that they overlap
    // the kernels on the caller's stream. Per group: V first (the mask build needs nothing else), then K and Q, then dO;
    // O and lse go back while the group's backward runs, the gradients while the next group computes. Events order the
    // helpers after the work already on the caller's stream and the caller's stream after the last copy.
    enum { kV, kKQ, kdO, kO, kG, kPerGroup };
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_done = nullptr;
    cudaEvent_t ev[kMaxGroups * kPerGroup] = {};
    auto cleanup = [&](int code) {
        for (int i = 0; i < NG * kPerGroup; ++i) if (ev[i]) cudaEventDestroy(ev[i]);
        if (ev_start) cudaEventDestroy(ev_start);
        if (ev_done) cudaEventDestroy(ev_done);
        if (s_in) cudaStreamDestroy(s_in);
        if (s_out) cudaStreamDestroy(s_out);
        return code;
    };
    if (cudaStreamCreateWithFlags(&s_in, cudaStreamNonBlocking) != cudaSuccess) return cleanup(DMA_ERR_CUDA);
    if (cudaStreamCreateWithFlags(&s_out, cudaStreamNonBlocking) != cudaSuccess) return cleanup(DMA_ERR_CUDA);
    if (cudaEventCreateWithFlags(&ev_start, cudaEventDisableTiming) != cudaSuccess) return cleanup(DMA_ERR_CUDA);
    if (cudaEventCreateWithFlags(&ev_done, cudaEventDisableTiming) != cudaSuccess) return cleanup(DMA_ERR_CUDA);
    for (int i = 0; i < NG * kPerGroup; ++i)
        if (cudaEventCreateWithFlags(&ev[i], cudaEventDisableTiming) != cudaSuccess) return cleanup(DMA_ERR_CUDA);

    // a [rows x width] block of a [rows x pitch] tensor; width == pitch is one plain copy
    auto copy2d = [&](void* dst, const void* src, size_t pitch, size_t width, size_t rows, cudaMemcpyKind kind, cudaStream_t on) {
        if (width == pitch) return cudaMemcpyAsync(dst, src, width * rows, kind, on) == cudaSuccess;
        return cudaMemcpy2DAsync(dst, pitch, src, pitch, width, rows, kind, on) == cudaSuccess;
    };
    auto rec = [&](cudaEvent_t e, cudaStream_t on) { return cudaEventRecord(e, on) == cudaSuccess; };
    auto wait = [&](cudaStream_t on, cudaEvent_t e) { return cudaStreamWaitEvent(on, e, 0) == cudaSuccess; };

    struct Group { size_t q, k, h; int hq0; };
    auto group_of = [&](int g) {
        const int b = g / HG, hg = g % HG;
        Group G;
        G.hq0 = hg * nqh;
        G.q = ((size_t)b * L * p->Hq + (size_t)hg * nqh) * d;          // elements into Q, O, dO, dQ
        G.k = ((size_t)b * L * p->Hkv + (size_t)hg * nkh) * d;         // elements into K, V, dK, dV
        G.h = ((size_t)b * p->Hq + (size_t)hg * nqh) * L;              // entries into the host's lse and dM
        return G;
    };
    const size_t q_pitch = (size_t)p->Hq * d * esz, q_width = (size_t)nqh * d * esz;
    const size_t k_pitch = (size_t)p->Hkv * d * esz, k_width = (size_t)nkh * d * esz;

    bool ok = rec(ev_start, st) && wait(s_in, ev_start) && wait(s_out, ev_start);
    ok = ok && cudaMemcpyAsync(a + Lo.W, hW_delta, Lo.wbytes, cudaMemcpyHostToDevice, s_in) == cudaSuccess &&
         cudaMemcpyAsync(a + Lo.A, hA, (size_t)p->Hq * 4, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
    for (int g = 0; g < NG && ok; ++g) {
        const Group G = group_of(g);
        cudaEvent_t* e = ev + g * kPerGroup;
        const cudaMemcpyKind in = cudaMemcpyHostToDevice;
        ok = copy2d(a + Lo.V + G.k * esz, (const char*)hV + G.k * esz, k_pitch, k_width, rows, in, s_in) && rec(e[kV], s_in) &&
             copy2d(a + Lo.K + G.k * esz, (const char*)hK + G.k * esz, k_pitch, k_width, rows, in, s_in) &&
             copy2d(a + Lo.Q + G.q * esz, (const char*)hQ + G.q * esz, q_pitch, q_width, rows, in, s_in) && rec(e[kKQ], s_in);
        if (backward) ok = ok && copy2d(a + Lo.dO + G.q * esz, (const char*)hdO + G.q * esz, q_pitch, q_width, rows, in, s_in) && rec(e[kdO], s_in);
    }
    if (!ok) return cleanup(DMA_ERR_CUDA);

    dma_problem_t sub = *p;
    sub.B = GB; sub.Hq = nqh; sub.Hkv = nkh;
    const int64_t qs[3] = {(int64_t)L * p->Hq * d, (int64_t)p->Hq * d, d}, ks[3] = {(int64_t)L * p->Hkv * d, (int64_t)p->Hkv * d, d};
    for (int i = 0; i < 3; ++i) { sub.q_stride[i] = sub.o_stride[i] = qs[i]; sub.k_stride[i] = sub.v_stride[i] = ks[i]; }
    const size_t f_ws = Lo.f_ws - (size_t)NG * kWsHeaderBytes, b_ws = Lo.b_ws - (size_t)NG * kWsHeaderBytes;
    const size_t w_per_head = Lo.wbytes / 4 / p->Hq;
    for (int g = 0; g < NG; ++g) {
        const Group G = group_of(g);
        cudaEvent_t* e = ev + g * kPerGroup;
        float* bias = (float*)(a + Lo.bias) + (size_t)g * Lo.gh;
        int32_t* expiry = (int32_t*)(a + Lo.expiry) + (size_t)g * Lo.gh;
        uint32_t* bitmap = (uint32_t*)(a + Lo.bitmap) + (size_t)g * Lo.gbmp;
        float* lse = (float*)(a + Lo.lse) + (size_t)g * Lo.gh;
        char* wsf = a + Lo.ws_fwd + (size_t)g * kWsHeaderBytes;
        if (!wait(st, e[kV])) return cleanup(DMA_ERR_CUDA);
        if ((rc = dma_mask_build(&sub, a + Lo.V + G.k * esz, (float*)(a + Lo.W) + G.hq0 * w_per_head, (float*)(a + Lo.A) + G.hq0, bias,
                                 expiry, bitmap, a + Lo.ws_mask, Lo.m_ws, st))) return cleanup(rc);
        if (!wait(st, e[kKQ])) return cleanup(DMA_ERR_CUDA);
        if ((rc = dma_attn_fwd(&sub, a + Lo.Q + G.q * esz, a + Lo.K + G.k * esz, a + Lo.V + G.k * esz, bias, expiry, bitmap,
                               a + Lo.O + G.q * esz, lse, wsf, f_ws, st))) return cleanup(rc);
        const cudaMemcpyKind out = cudaMemcpyDeviceToHost;
        ok = rec(e[kO], st) && wait(s_out, e[kO]) &&
             copy2d((char*)hO + G.q * esz, a + Lo.O + G.q * esz, q_pitch, q_width, rows, out, s_out) &&
             cudaMemcpyAsync(hlse + G.h, lse, hl * 4, out, s_out) == cudaSuccess;
        if (backward) {
            char* wsb = a + Lo.ws_bwd + (size_t)g * kWsHeaderBytes;
            float* dM = (float*)(a + Lo.dM) + (size_t)g * Lo.gh;
            if (!ok || !wait(st, e[kdO])) return cleanup(DMA_ERR_CUDA);
            if ((rc = dma_attn_bwd(&sub, a + Lo.Q + G.q * esz, a + Lo.K + G.k * esz, a + Lo.V + G.k * esz, a + Lo.O + G.q * esz,
                                   a + Lo.dO + G.q * esz, lse, bias, expiry, bitmap, a + Lo.dQ + G.q * esz, a + Lo.dK + G.k * esz,
                                   a + Lo.dV + G.k * esz, dM, wsb, b_ws, st))) return cleanup(rc);
            ok = rec(e[kG], st) && wait(s_out, e[kG]) &&
                 copy2d((char*)hdQ + G.q * esz, a + Lo.dQ + G.q * esz, q_pitch, q_width, rows, out, s_out) &&
                 copy2d((char*)hdK + G.k * esz, a + Lo.dK + G.k * esz, k_pitch, k_width, rows, out, s_out) &&
                 copy2d((char*)hdV + G.k * esz, a + Lo.dV + G.k * esz, k_pitch, k_width, rows, out, s_out) &&
                 cudaMemcpyAsync(hdM + G.h, dM, hl * 4, out, s_out) == cudaSuccess;
        }
        if (!ok) return cleanup(DMA_ERR_CUDA);
    }
    ok = rec(ev_done, s_out) && wait(st, ev_done);
    if (!ok) return cleanup(DMA_ERR_CUDA);
    if (cudaStreamSynchronize(st) != cudaSuccess) return cleanup(DMA_ERR_CUDA);
    // the groups' status words (one header each in front of the forward and of the backward workspace)
    static_assert(kWsHeaderBytes % 4 == 0, "header");
    int32_t heads[kMaxGroups * (kWsHeaderBytes / 4)];
    for (int pass = 0; pass < (backward ? 2 : 1); ++pass) {
        const char* src = a + (pass ? Lo.ws_bwd : Lo.ws_fwd);
        if (cudaMemcpyAsync(heads, src, (size_t)NG * kWsHeaderBytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return cleanup(DMA_ERR_CUDA);
        if (cudaStreamSynchronize(st) != cudaSuccess) return cleanup(DMA_ERR_CUDA);
        for (int g = 0; g < NG; ++g)
            if (heads[g * (kWsHeaderBytes / 4)] != 0) return cleanup(DMA_ERR_DEVICE_TIMEOUT);
    }
    return cleanup(DMA_OK);
}

}  // extern "C"
