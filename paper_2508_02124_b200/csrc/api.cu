// C-ABI entry points (include/dma.h): argument validation, defaults, dispatch to the stage launchers.
#include <atomic>
#include <cmath>
#include <mutex>
#include <vector>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace dma {

static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches += n; }
int check_launch() { return cudaGetLastError() == cudaSuccess ? DMA_OK : DMA_ERR_CUDA; }

// ---- dma_kernel_timing: event pairs around the main kernel of each attention call while recording is on ----------
namespace {
struct TimedLaunch { cudaEvent_t before, after; int which; bool closed; };
constexpr size_t kMaxTimed = 4096;
std::mutex g_timing_mutex;
std::vector<TimedLaunch> g_timed;
std::atomic<bool> g_timing_on{false};
void timing_clear() {
    for (TimedLaunch& t : g_timed) { cudaEventDestroy(t.before); cudaEventDestroy(t.after); }
    g_timed.clear();
}
}  // namespace

void timing_mark(int which, bool after, cudaStream_t st) {
    if (!g_timing_on.load(std::memory_order_relaxed)) return;
    std::lock_guard<std::mutex> lock(g_timing_mutex);
    if (!after) {
        if (g_timed.size() >= kMaxTimed) return;
        TimedLaunch t{nullptr, nullptr, which, false};
        if (cudaEventCreate(&t.before) != cudaSuccess) return;
        if (cudaEventCreate(&t.after) != cudaSuccess) { cudaEventDestroy(t.before); return; }
        cudaEventRecord(t.before, st);
        g_timed.push_back(t);
    } else if (!g_timed.empty() && !g_timed.back().closed && g_timed.back().which == which) {
        cudaEventRecord(g_timed.back().after, st);
        g_timed.back().closed = true;
    }
}

static bool fill_strides(const int64_t in[3], int64_t out[3], int L, int H, int d) {
    if (in[0] == 0 && in[1] == 0 && in[2] == 0) {
        out[0] = (int64_t)L * H * d; out[1] = (int64_t)H * d; out[2] = d;
        return true;
    }
    for (int i = 0; i < 3; ++i) {
        if (in[i] <= 0 || in[i] % 8) return false;
        out[i] = in[i];
    }
    return true;
}

int resolve(const dma_problem_t* p, Prob* o) {
    if (!p) return DMA_ERR_NULL;
    if (p->B < 1 || p->Hq < 1 || p->Hkv < 1 || p->L < 1 || p->w < 1 || p->Hq % p->Hkv) return DMA_ERR_SHAPE;
    if (p->d != 64 && p->d != 128) return DMA_ERR_UNSUPPORTED;
    if (p->causal != 0 && p->causal != 1) return DMA_ERR_UNSUPPORTED;
    if (p->dtype != DMA_BF16 && p->dtype != DMA_FP32) return DMA_ERR_UNSUPPORTED;
    if ((p->tile_m == 0) != (p->tile_n == 0) || p->tile_m < 0 || p->tile_n < 0) return DMA_ERR_SHAPE;
    if (!(p->softmax_scale >= 0.0f) || std::isinf(p->softmax_scale)) return DMA_ERR_SHAPE;
    o->B = p->B; o->Hq = p->Hq; o->Hkv = p->Hkv; o->L = p->L; o->d = p->d; o->G = p->Hq / p->Hkv;
    o->w = p->w < p->L ? p->w : p->L;
    o->w_cap = p->w;
    o->Lq = p->L; o->q_off = 0;
    o->dtype = p->dtype; o->flags = p->flags; o->causal = p->causal;
    o->bm = p->tile_m ? p->tile_m : 128;
    o->bn = p->tile_n ? p->tile_n : 128;
    o->Tr = (p->L + o->bm - 1) / o->bm;
    o->Tc = (p->L + o->bn - 1) / o->bn;
    o->Wd = (o->Tc + 31) / 32;
    o->scale = p->softmax_scale > 0.0f ? p->softmax_scale : 1.0f / sqrtf((float)p->d);
    if (!fill_strides(p->q_stride, o->qs, p->L, p->Hq, p->d) || !fill_strides(p->k_stride, o->ks, p->L, p->Hkv, p->d) ||
        !fill_strides(p->v_stride, o->vs, p->L, p->Hkv, p->d) || !fill_strides(p->o_stride, o->os, p->L, p->Hq, p->d))
        return DMA_ERR_ALIGN;
    const bool tc_shape = o->dtype == DMA_BF16 && o->bm == 128 && o->bn == 128 && !(o->flags & DMA_FLAG_SIMT);
    if (o->flags & DMA_FLAG_IGNORE_BITMAP) o->flags |= DMA_FLAG_TILE_PATH;
    if ((o->flags & DMA_FLAG_TILE_PATH) && (o->flags & DMA_FLAG_COMPACT_KV)) return DMA_ERR_UNSUPPORTED;
    if (!o->causal && tc_shape) {
        // non-causal: all rows of a head keep the same keys, so the tensor-core path always runs token-compacted
        if (o->flags & DMA_FLAG_TILE_PATH) return DMA_ERR_UNSUPPORTED;
        o->flags |= DMA_FLAG_COMPACT_KV;
    } else if (tc_shape && !(o->flags & (DMA_FLAG_COMPACT_KV | DMA_FLAG_TILE_PATH)) && o->L >= 2048 && 4ll * o->w <= o->L) {
        // the library's choice (a function of the descriptor alone): with a window of at most a quarter of the
        // sequence the token-compacted kernels do O(L w d) work where walking tiles does O(L^2 d) on scattered masks
        o->flags |= DMA_FLAG_COMPACT_KV;
    }
    return DMA_OK;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

static bool use_tensor_cores(const Prob& P) {
    return P.dtype == DMA_BF16 && (P.d == 128 || P.d == 64) && P.bm == 128 && P.bn == 128 && !(P.flags & DMA_FLAG_SIMT);
}

static size_t fwd_ws_any(const Prob& P) { return use_tensor_cores(P) ? tc_fwd_ws_bytes(P) : (size_t)kWsHeaderBytes; }

static size_t bwd_ws_any(const Prob& P) { return use_tensor_cores(P) ? tc_bwd_ws_bytes(P) : simt_bwd_ws_bytes(P); }

static int fwd_any(const Prob& P, const void* Q, const void* K, const void* V, const float* bias, const int32_t* expiry,
                   const uint32_t* bitmap, void* O, float* lse, void* ws, cudaStream_t st) {
    if (use_tensor_cores(P)) return launch_tc_fwd(P, Q, K, V, bias, expiry, bitmap, O, lse, ws, st);
    return launch_simt_fwd(P, Q, K, V, bias, expiry, bitmap, O, lse, st);
}

static int bwd_any(const Prob& P, const void* Q, const void* K, const void* V, const void* O, const void* dO, const float* lse,
                   const float* bias, const int32_t* expiry, const uint32_t* bitmap, void* dQ, void* dK, void* dV, float* dM,
                   void* ws, cudaStream_t st) {
    if (use_tensor_cores(P)) return launch_tc_bwd(P, Q, K, V, O, dO, lse, bias, expiry, bitmap, dQ, dK, dV, dM, ws, st);
    return launch_simt_bwd(P, Q, K, V, O, dO, lse, bias, expiry, bitmap, dQ, dK, dV, dM, ws, st);
}

static int device_ok() {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return DMA_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return DMA_ERR_CUDA;
    return major == 10 ? DMA_OK : DMA_ERR_CUDA;
}

// One CTA waits on an mbarrier that nothing ever arrives at, with a limit of about two milliseconds: the wait gives
// up, the abort flag is raised and the status word is written, exactly as in the attention kernels.
__global__ void selftest_wait_kernel(int32_t* status) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        abort_flag = 0;
        ptx::fence_barrier_init();
    }
    __syncthreads();
    const bool ok = ptx::mbar_wait(&bar, 0, &abort_flag, 1ll << 22);
    __syncthreads();
    if (threadIdx.x == 0 && (!ok || abort_flag)) atomicExch(status, (int32_t)DMA_ERR_DEVICE_TIMEOUT);
}

}  // namespace dma

using namespace dma;

extern "C" {

int dma_query_workspace(const dma_problem_t* p, size_t* mask_ws, size_t* fwd_ws, size_t* bwd_ws) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    if (mask_ws) *mask_ws = mask_ws_bytes(P);
    if (fwd_ws) *fwd_ws = fwd_ws_any(P);
    if (bwd_ws) *bwd_ws = bwd_ws_any(P);
    return DMA_OK;
}

int dma_bitmap_words(const dma_problem_t* p, size_t* words) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    if (!words) return DMA_ERR_NULL;
    *words = (size_t)P.B * P.Hq * P.Tr * P.Wd;
    return DMA_OK;
}

int dma_mask_build(const dma_problem_t* p, const void* V, const float* W_delta, const float* A, float* bias,
                   int32_t* expiry, uint32_t* bitmap, void* ws, size_t ws_bytes, void* cuda_stream) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    if (!V || !W_delta || !A || !bias || !expiry || !bitmap) return DMA_ERR_NULL;
    if (!aligned16(V) || !aligned16(W_delta) || !aligned16(bias) || !aligned16(expiry) || !aligned16(bitmap))
        return DMA_ERR_ALIGN;
    if (!ws || ws_bytes < mask_ws_bytes(P) || !aligned16(ws)) return DMA_ERR_WORKSPACE;
    if ((rc = device_ok())) return rc;
    return launch_mask_build(P, V, W_delta, A, bias, expiry, bitmap, ws, (cudaStream_t)cuda_stream);
}

int dma_mask_build_varlen(const dma_problem_t* p, const void* V, const float* W_delta, const float* A,
                          const int32_t* cu_seqlens, int32_t nseq, float* bias, int32_t* expiry, uint32_t* bitmap,
                          void* ws, size_t ws_bytes, void* cuda_stream) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    if (!V || !W_delta || !A || !cu_seqlens || !bias || !expiry || !bitmap) return DMA_ERR_NULL;
    if (nseq < 1 || nseq > P.L) return DMA_ERR_SHAPE;
    if (!P.causal) return DMA_ERR_UNSUPPORTED;
    if (!aligned16(V) || !aligned16(W_delta) || !aligned16(bias) || !aligned16(expiry) || !aligned16(bitmap))
        return DMA_ERR_ALIGN;
    if (!ws || ws_bytes < mask_ws_bytes(P) || !aligned16(ws)) return DMA_ERR_WORKSPACE;
    if ((rc = device_ok())) return rc;
    return launch_mask_build(P, V, W_delta, A, bias, expiry, bitmap, ws, (cudaStream_t)cuda_stream, cu_seqlens, nseq);
}

int dma_mask_bwd_workspace(const dma_problem_t* p, size_t* bytes) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    if (!bytes) return DMA_ERR_NULL;
    *bytes = mask_bwd_ws_bytes(P);
    return DMA_OK;
}

int dma_mask_bwd(const dma_problem_t* p, const void* V, const float* W_delta, const float* A, const float* bias,
                 const float* dM, void* dV, float* dW_delta, float* dA, void* ws, size_t ws_bytes, void* cuda_stream) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    if (!V || !W_delta || !A || !bias || !dM || !dV || !dW_delta || !dA) return DMA_ERR_NULL;
    if (!aligned16(V) || !aligned16(W_delta) || !aligned16(bias) || !aligned16(dM) || !aligned16(dV) || !aligned16(dW_delta))
        return DMA_ERR_ALIGN;
    if (!ws || ws_bytes < mask_bwd_ws_bytes(P) || !aligned16(ws)) return DMA_ERR_WORKSPACE;
    if ((rc = device_ok())) return rc;
    return launch_mask_bwd(P, V, W_delta, A, bias, dM, dV, dW_delta, dA, ws, (cudaStream_t)cuda_stream);
}

int dma_delta_range(const dma_problem_t* p, const void* V, const float* W_delta, const float* A, float* delta, int64_t delta_ld,
                    int32_t j_begin, int32_t j_end, void* cuda_stream) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    if (!V || !W_delta || !A || !delta) return DMA_ERR_NULL;
    if (!aligned16(V) || !aligned16(W_delta) || !aligned16(delta)) return DMA_ERR_ALIGN;
    if (j_begin < 0 || j_end > P.L || j_begin > j_end || delta_ld < P.L) return DMA_ERR_SHAPE;
    if ((rc = device_ok())) return rc;
    return launch_delta_range(P, V, W_delta, A, delta, delta_ld, j_begin, j_end, (cudaStream_t)cuda_stream);
}

int dma_decode_workspace(const dma_problem_t* p, size_t* bytes) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    if (!bytes) return DMA_ERR_NULL;
    *bytes = decode_ws_bytes(P);
    return DMA_OK;
}

int dma_decode(const dma_problem_t* p, const void* q, const void* K, const void* V, const float* delta, int64_t delta_ld,
               void* o, float* lse, int32_t* sel_idx, void* ws, size_t ws_bytes, void* cuda_stream) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    if (!q || !K || !V || !delta || !o || !lse) return DMA_ERR_NULL;
    if (!aligned16(q) || !aligned16(K) || !aligned16(V) || !aligned16(delta) || !aligned16(o)) return DMA_ERR_ALIGN;
    if (delta_ld < P.L) return DMA_ERR_SHAPE;
    if (!ws || ws_bytes < decode_ws_bytes(P) || !aligned16(ws)) return DMA_ERR_WORKSPACE;
    if ((rc = device_ok())) return rc;
    return launch_decode(P, q, K, V, delta, delta_ld, o, lse, sel_idx, ws, (cudaStream_t)cuda_stream);
}

int dma_decode_state_bytes(const dma_problem_t* p, size_t* bytes) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    if (!bytes) return DMA_ERR_NULL;
    *bytes = decode_state_bytes(P);
    return DMA_OK;
}

int dma_decode_state_init(const dma_problem_t* p, const float* delta, int64_t delta_ld, void* state, void* ws, size_t ws_bytes,
                          void* cuda_stream) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    if (!delta || !state) return DMA_ERR_NULL;
    if (!aligned16(delta) || !aligned16(state)) return DMA_ERR_ALIGN;
    if (delta_ld < P.L) return DMA_ERR_SHAPE;
    if (!ws || ws_bytes < decode_ws_bytes(P) || !aligned16(ws)) return DMA_ERR_WORKSPACE;
    if ((rc = device_ok())) return rc;
    return launch_decode_state_init(P, delta, delta_ld, (int*)state, ws, (cudaStream_t)cuda_stream);
}

int dma_decode_step(const dma_problem_t* p, const void* q, const void* K, const void* V, const float* delta, int64_t delta_ld,
                    void* state, void* o, float* lse, void* ws, size_t ws_bytes, void* cuda_stream) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    if (!q || !K || !V || !delta || !state || !o || !lse) return DMA_ERR_NULL;
    if (!aligned16(q) || !aligned16(K) || !aligned16(V) || !aligned16(delta) || !aligned16(state) || !aligned16(o)) return DMA_ERR_ALIGN;
    if (delta_ld < P.L) return DMA_ERR_SHAPE;
    if (!ws || ws_bytes < decode_ws_bytes(P) || !aligned16(ws)) return DMA_ERR_WORKSPACE;
    if ((rc = device_ok())) return rc;
    return launch_decode_step(P, q, K, V, delta, delta_ld, (int*)state, o, lse, ws, (cudaStream_t)cuda_stream);
}

int dma_attn_fwd(const dma_problem_t* p, const void* Q, const void* K, const void* V, const float* bias,
                 const int32_t* expiry, const uint32_t* bitmap, void* O, float* lse, void* ws, size_t ws_bytes,
                 void* cuda_stream) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    if (!Q || !K || !V || !bias || !expiry || !bitmap || !O || !lse) return DMA_ERR_NULL;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(bias) || !aligned16(expiry) ||
        !aligned16(lse))
        return DMA_ERR_ALIGN;
    const bool tc = use_tensor_cores(P);
    if ((P.flags & DMA_FLAG_COMPACT_KV) && !tc) return DMA_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < fwd_ws_any(P) || !aligned16(ws)) return DMA_ERR_WORKSPACE;
    if ((rc = device_ok())) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(ws, 0, kWsHeaderBytes, st) != cudaSuccess) return DMA_ERR_CUDA;
    return fwd_any(P, Q, K, V, bias, expiry, bitmap, O, lse, ws, st);
}

int dma_attn_fwd_chunk(const dma_problem_t* p, int32_t q_begin, int32_t q_len, const void* Q, const void* K, const void* V,
                       const float* bias, const int32_t* expiry, void* O, float* lse, void* ws, size_t ws_bytes,
                       void* cuda_stream) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    if (!Q || !K || !V || !bias || !expiry || !O || !lse) return DMA_ERR_NULL;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(bias) || !aligned16(expiry) ||
        !aligned16(lse))
        return DMA_ERR_ALIGN;
    if (q_begin < 0 || q_len < 1 || (int64_t)q_begin + q_len > P.L) return DMA_ERR_SHAPE;
    P.Lq = q_len; P.q_off = q_begin;
    bool q_default = true, o_default = true;
    for (int t = 0; t < 3; ++t) { q_default = q_default && p->q_stride[t] == 0; o_default = o_default && p->o_stride[t] == 0; }
    const int64_t packed[3] = {(int64_t)q_len * P.Hq * P.d, (int64_t)P.Hq * P.d, P.d};     // [B, q_len, Hq, d]
    for (int t = 0; t < 3; ++t) {
        if (q_default) P.qs[t] = packed[t];
        if (o_default) P.os[t] = packed[t];
    }
    if (use_tensor_cores(P)) P.flags |= DMA_FLAG_COMPACT_KV;   // the gathered-key kernel has no tile alignment between rows and keys
    if (!ws || ws_bytes < fwd_ws_any(P) || !aligned16(ws)) return DMA_ERR_WORKSPACE;
    if ((rc = device_ok())) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(ws, 0, kWsHeaderBytes, st) != cudaSuccess) return DMA_ERR_CUDA;
    return fwd_any(P, Q, K, V, bias, expiry, nullptr, O, lse, ws, st);
}

int dma_attn_bwd(const dma_problem_t* p, const void* Q, const void* K, const void* V, const void* O, const void* dO,
                 const float* lse, const float* bias, const int32_t* expiry, const uint32_t* bitmap, void* dQ, void* dK,
                 void* dV, float* dM, void* ws, size_t ws_bytes, void* cuda_stream) {
    Prob P;
    int rc = resolve(p, &P);
    if (rc) return rc;
    if (!Q || !K || !V || !O || !dO || !lse || !bias || !expiry || !bitmap || !dQ || !dK || !dV || !dM) return DMA_ERR_NULL;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(dO) || !aligned16(dQ) ||
        !aligned16(dK) || !aligned16(dV) || !aligned16(dM) || !aligned16(lse))
        return DMA_ERR_ALIGN;
    const bool tc = use_tensor_cores(P);
    if ((P.flags & DMA_FLAG_COMPACT_KV) && !tc) return DMA_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < bwd_ws_any(P) || !aligned16(ws)) return DMA_ERR_WORKSPACE;
    if ((rc = device_ok())) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(ws, 0, kWsHeaderBytes, st) != cudaSuccess) return DMA_ERR_CUDA;
    return bwd_any(P, Q, K, V, O, dO, lse, bias, expiry, bitmap, dQ, dK, dV, dM, ws, st);
}

int dma_read_status(const void* ws, void* cuda_stream) {
    if (!ws) return DMA_ERR_NULL;
    int32_t word = 0;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess) return DMA_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return DMA_ERR_CUDA;
    return word == 0 ? DMA_OK : word == DMA_ERR_MASK_OVERFLOW ? DMA_ERR_MASK_OVERFLOW : DMA_ERR_DEVICE_TIMEOUT;
}

int dma_selftest_wait_timeout(void* ws, size_t ws_bytes, void* cuda_stream) {
    if (!ws || ws_bytes < (size_t)kWsHeaderBytes || !aligned16(ws)) return DMA_ERR_WORKSPACE;
    int rc = device_ok();
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(ws, 0, kWsHeaderBytes, st) != cudaSuccess) return DMA_ERR_CUDA;
    selftest_wait_kernel<<<1, 64, 0, st>>>((int32_t*)ws);
    count_launch();
    return check_launch();
}

long long dma_launch_count(void) { return g_launches.load(); }

int dma_kernel_timing(int enable) {
    std::lock_guard<std::mutex> lock(g_timing_mutex);
    if (enable) timing_clear();
    g_timing_on.store(enable != 0);
    return DMA_OK;
}

int dma_kernel_timing_read(float* ms, int32_t* which, int32_t capacity, int32_t* count) {
    if (!count || (capacity > 0 && (!ms || !which))) return DMA_ERR_NULL;
    std::lock_guard<std::mutex> lock(g_timing_mutex);
    int n = 0;
    for (const TimedLaunch& t : g_timed) {
        if (!t.closed) continue;
        if (n < capacity) {
            if (cudaEventSynchronize(t.after) != cudaSuccess || cudaEventElapsedTime(&ms[n], t.before, t.after) != cudaSuccess)
                return DMA_ERR_CUDA;
            which[n] = t.which;
        }
        ++n;
    }
    *count = n;
    return DMA_OK;
}

const char* dma_strerror(int status) {
    switch (status) {
        case DMA_OK: return "ok";
        case DMA_ERR_NULL: return "a required pointer is NULL";
        case DMA_ERR_SHAPE: return "invalid shape, window, tile size or scale";
        case DMA_ERR_ALIGN: return "pointer not 16-byte aligned or stride not a positive multiple of 8 elements";
        case DMA_ERR_UNSUPPORTED: return "request outside the implemented range (d in {64,128}, causal=1, bf16/fp32)";
        case DMA_ERR_WORKSPACE: return "workspace missing, misaligned or smaller than dma_query_workspace reports";
        case DMA_ERR_CUDA: return "CUDA call failed or no sm_100 device";
        case DMA_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
        case DMA_ERR_MASK_OVERFLOW: return "token-compacted execution: the mask keeps more than w keys in a row";
        default: return "unknown status";
    }
}

}  // extern "C"
