// dma_step_host: the whole hot path (mask build, forward, optional backward) on HOST buffers, for callers that
// keep their tensors in host memory and for end-to-end timing. Inputs are copied to a caller-provided device
// arena (on helper streams, overlapped with the kernels), the three stages run on the caller's stream, results are
// copied back, and the stream is synchronised.
#include "common.cuh"

namespace dma {
namespace {

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
};

int make_layout(const dma_problem_t* p, int backward, Layout* Lo) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    for (int i = 0; i < 3; ++i)
        if (p->q_stride[i] || p->k_stride[i] || p->v_stride[i] || p->o_stride[i]) return DMA_ERR_UNSUPPORTED;
    if ((rc = dma_query_workspace(p, &Lo->m_ws, &Lo->f_ws, &Lo->b_ws))) return rc;
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
    Lo->bias = a.take(Lo->nbh * 4); Lo->expiry = a.take(Lo->nbh * 4); Lo->bitmap = a.take(Lo->nbmp * 4);
    Lo->lse = a.take(Lo->nbh * 4);
    Lo->ws_mask = a.take(Lo->m_ws); Lo->ws_fwd = a.take(Lo->f_ws);
    if (backward) {
        Lo->dO = a.take(Lo->nq * Lo->esz); Lo->dQ = a.take(Lo->nq * Lo->esz);
        Lo->dK = a.take(Lo->nk * Lo->esz); Lo->dV = a.take(Lo->nk * Lo->esz);
        Lo->dM = a.take(Lo->nbh * 4); Lo->ws_bwd = a.take(Lo->b_ws);
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
    // Copies run on two helper streams of this call (created and destroyed here: no state is kept) so that they overlap
    // the kernels on the caller's stream: V first (the mask build needs nothing else), then K and Q, then dO while the
    // forward runs; O and lse go back while the backward runs. Events order the helpers after the work already on the
    // caller's stream and the caller's stream after the last copy.
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev[7] = {};
    auto cleanup = [&](int code) {
        for (auto& e : ev) if (e) cudaEventDestroy(e);
        if (s_in) cudaStreamDestroy(s_in);
        if (s_out) cudaStreamDestroy(s_out);
        return code;
    };
    if (cudaStreamCreateWithFlags(&s_in, cudaStreamNonBlocking) != cudaSuccess) return cleanup(DMA_ERR_CUDA);
    if (cudaStreamCreateWithFlags(&s_out, cudaStreamNonBlocking) != cudaSuccess) return cleanup(DMA_ERR_CUDA);
    for (auto& e : ev) if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return cleanup(DMA_ERR_CUDA);
    enum { kStart, kV, kKQ, kdO, kO, kG, kDone };
    auto h2d = [&](size_t off, const void* src, size_t n) { return cudaMemcpyAsync(a + off, src, n, cudaMemcpyHostToDevice, s_in) == cudaSuccess; };
    auto d2h = [&](void* dst, size_t off, size_t n) { return cudaMemcpyAsync(dst, a + off, n, cudaMemcpyDeviceToHost, s_out) == cudaSuccess; };
    auto rec = [&](int e, cudaStream_t on) { return cudaEventRecord(ev[e], on) == cudaSuccess; };
    auto wait = [&](cudaStream_t on, int e) { return cudaStreamWaitEvent(on, ev[e], 0) == cudaSuccess; };
    bool ok = rec(kStart, st) && wait(s_in, kStart) && wait(s_out, kStart);
    ok = ok && h2d(Lo.V, hV, Lo.nk * Lo.esz) && h2d(Lo.W, hW_delta, Lo.wbytes) && h2d(Lo.A, hA, (size_t)p->Hq * 4) && rec(kV, s_in);
    ok = ok && h2d(Lo.K, hK, Lo.nk * Lo.esz) && h2d(Lo.Q, hQ, Lo.nq * Lo.esz) && rec(kKQ, s_in);
    if (backward) ok = ok && h2d(Lo.dO, hdO, Lo.nq * Lo.esz) && rec(kdO, s_in);
    if (!ok) return cleanup(DMA_ERR_CUDA);
    float* bias = (float*)(a + Lo.bias);
    int32_t* expiry = (int32_t*)(a + Lo.expiry);
    uint32_t* bitmap = (uint32_t*)(a + Lo.bitmap);
    if (!wait(st, kV)) return cleanup(DMA_ERR_CUDA);
    if ((rc = dma_mask_build(p, a + Lo.V, (float*)(a + Lo.W), (float*)(a + Lo.A), bias, expiry, bitmap, a + Lo.ws_mask, Lo.m_ws, st))) return cleanup(rc);
    if (!wait(st, kKQ)) return cleanup(DMA_ERR_CUDA);
    if ((rc = dma_attn_fwd(p, a + Lo.Q, a + Lo.K, a + Lo.V, bias, expiry, bitmap, a + Lo.O, (float*)(a + Lo.lse), a + Lo.ws_fwd, Lo.f_ws, st))) return cleanup(rc);
    ok = rec(kO, st) && wait(s_out, kO) && d2h(hO, Lo.O, Lo.nq * Lo.esz) && d2h(hlse, Lo.lse, Lo.nbh * 4);
    if (backward) {
        if (!ok || !wait(st, kdO)) return cleanup(DMA_ERR_CUDA);
        if ((rc = dma_attn_bwd(p, a + Lo.Q, a + Lo.K, a + Lo.V, a + Lo.O, a + Lo.dO, (float*)(a + Lo.lse), bias, expiry, bitmap,
                               a + Lo.dQ, a + Lo.dK, a + Lo.dV, (float*)(a + Lo.dM), a + Lo.ws_bwd, Lo.b_ws, st))) return cleanup(rc);
        ok = rec(kG, st) && wait(s_out, kG) && d2h(hdQ, Lo.dQ, Lo.nq * Lo.esz) && d2h(hdK, Lo.dK, Lo.nk * Lo.esz) &&
             d2h(hdV, Lo.dV, Lo.nk * Lo.esz) && d2h(hdM, Lo.dM, Lo.nbh * 4);
    }
    ok = ok && rec(kDone, s_out) && wait(st, kDone);
    if (!ok) return cleanup(DMA_ERR_CUDA);
    if (cudaStreamSynchronize(st) != cudaSuccess) return cleanup(DMA_ERR_CUDA);
    int s1 = dma_read_status(a + Lo.ws_fwd, st);
    if (s1) return cleanup(s1);
    return cleanup(backward ? dma_read_status(a + Lo.ws_bwd, st) : DMA_OK);
}

}  // extern "C"
