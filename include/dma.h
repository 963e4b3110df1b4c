/* dma.h - C ABI of the B200 (sm_100a) Dynamic Mask Attention hot path.
 *
 * Three stages, each one entry point:
 *   dma_mask_build   value vectors -> per-key dynamic weight (the additive bias), per-key expiry row
 *                    (compact form of the per-row top-w mask) and a (query tile, key tile) activity bitmap
 *   dma_attn_fwd     block-sparse attention forward: O and the row log-sum-exp
 *   dma_attn_bwd     backward: dQ, dK, dV and dM (gradient of the mask bias)
 *
 * Conventions
 *   - Unless a parameter is marked HOST, every pointer is a DEVICE pointer owned by the caller, 16-byte
 *     aligned. The library allocates no device memory, enqueues work only on the caller's stream (a
 *     cudaStream_t passed as void*; NULL = default stream) and does not synchronise, except in
 *     dma_read_status and dma_step_host. What it keeps between calls is bookkeeping only: the process-wide
 *     launch counter behind dma_launch_count, and for dma_mask_build_static the fixed scratch array in the
 *     device image with its per-device address; no result depends on an earlier call.
 *   - Element type of Q,K,V,O,dO,dQ,dK,dV is `dtype` (bf16 or fp32). bias, lse, dM, W_delta, A are fp32.
 *   - Q,O,dO,dQ are [B, L, Hq, d]; K,V,dK,dV are [B, L, Hkv, d]; d is contiguous; the batch, sequence and
 *     head strides are given in elements in the problem descriptor (0 = contiguous default). bias, expiry,
 *     lse, dM are contiguous [B, Hq, L]. Query head h reads KV head h / (Hq / Hkv).
 *   - Every entry point returns 0 (DMA_OK) or a negative dma_status code; nothing is thrown across the ABI.
 *     On an error return no kernel has been launched. Outputs are fully overwritten (no pre-zeroing needed).
 *   - There is no CPU path: without a CUDA device of compute capability 10.x the calls return DMA_ERR_CUDA.
 *   - The calls that take a stream only enqueue work on it: they allocate nothing and do not synchronise, so they can be
 *     captured into a CUDA graph. Exceptions: dma_step_host, dma_read_status and dma_selftest_wait_timeout synchronise
 *     the stream, and the first dma_mask_build_static call on a device looks up a symbol address.
 */
#ifndef DMA_B200_H
#define DMA_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DMA_OK = 0,
    DMA_ERR_NULL = -1,           /* a required pointer is NULL                                      */
    DMA_ERR_SHAPE = -2,          /* non-positive size, Hq % Hkv != 0, w < 1, bad tile size          */
    DMA_ERR_ALIGN = -3,          /* pointer not 16-byte aligned or stride not a multiple of 8       */
    DMA_ERR_UNSUPPORTED = -4,    /* valid request outside what is implemented (see each call)       */
    DMA_ERR_WORKSPACE = -5,      /* workspace NULL or smaller than dma_query_workspace reports      */
    DMA_ERR_CUDA = -6,           /* a CUDA runtime / driver call failed (launch, descriptor, device)*/
    DMA_ERR_DEVICE_TIMEOUT = -7, /* a bounded device-side wait gave up (read via dma_read_status)    */
    DMA_ERR_MASK_OVERFLOW = -8   /* token-compacted execution met a mask that keeps more than w keys in a row: the
                                    gathered key lists are sized for w (read via dma_read_status; the outputs of
                                    that call are not valid)                                          */
} dma_status;

enum { DMA_BF16 = 0, DMA_FP32 = 1 };

/* flags */
enum {
    DMA_FLAG_IGNORE_BITMAP = 1,  /* visit every causal tile regardless of the bitmap (result must not change:
                                    block skipping is an optimisation only, Sec. 4.2 last paragraph)           */
    DMA_FLAG_SIMT = 2,           /* run the CUDA-core kernels also for bf16 (they always serve fp32)            */
    DMA_FLAG_COMPACT_KV = 4,     /* dma_attn_fwd and dma_attn_bwd, bf16: token-compacted
                                    execution (Sec. 3.3, computational sparsity: O(L w d) instead of O(L^2 d) work).
                                    Forward: each pair of query tiles gathers only the keys that one of its 256 rows
                                    keeps (at most w + 256) instead of walking every active 128-key tile. Backward: a CTA
                                    owns 128 keys of one query head that expire within the same band of rows (a
                                    lifetime-sorted permutation built per call) and walks only the query tiles between
                                    the first key and the last expiry; dK, dV are summed over the group in fp32. Same
                                    results up to rounding; needs the larger workspaces dma_query_workspace reports for
                                    it; ignores the bitmap. The mask must keep at most w keys per row, as every mask
                                    of dma_mask_build does (an injected mask that keeps more needs p->w raised to its
                                    largest per-row count: the gathered lists are sized w + 256; a list that overflows
                                    leaves DMA_ERR_MASK_OVERFLOW in the workspace status word).
                                    WITHOUT this flag and without DMA_FLAG_TILE_PATH the library chooses: causal bf16
                                    problems on the tensor-core kernels with L >= 2048 and 4 w <= L run token-compacted
                                    (there the tile-walking kernels spend most of their work on (row, key) pairs the mask
                                    drops; from w = L/2 on the tile-walking kernels are the faster ones), everything else
                                    walks tiles. The choice depends on the descriptor alone, so dma_query_workspace,
                                    dma_attn_fwd and dma_attn_bwd agree on it */
    DMA_FLAG_TILE_PATH = 16,     /* dma_attn_fwd and dma_attn_bwd: always walk the bitmap's active 128 x 128 tiles (Alg. 1 /
                                    Alg. 2 with block skipping), never the token-compacted kernels. For masks whose kept
                                    keys cluster (packed documents, banded importance) tile skipping alone can be the
                                    faster choice; DMA_FLAG_IGNORE_BITMAP and DMA_FLAG_SIMT imply it */
    DMA_FLAG_BLOCK_SKIP = 32,    /* dma_attn_fwd, tensor-core kernels: MMA-block skipping inside executed tiles (the finer
                                    granularity below the 128 x 128 tile: "if there are no active tokens in the MMA block,
                                    skip"). The P V product leaves out the 16-key blocks in which no key can be kept by the
                                    query tile's rows; P is exactly zero there, so O and lse are the same bits. Off by
                                    default: on the benchmark masks well under 5 % of the blocks of executed tiles are dead,
                                    and the bookkeeping costs the kernel more than the multiplications it saves */
    DMA_FLAG_DETERMINISTIC = 64, /* dma_attn_bwd with token-compacted execution: the query heads of a group write their dK / dV
                                    contributions to accumulators of their own (Hq/Hkv times the accumulator space: the
                                    larger workspace dma_query_workspace reports) and a last pass adds them in head order,
                                    so dK and dV are the same bits from run to run, as on the tile path. dQ stays a sum of
                                    floating-point atomics on every path */
    DMA_FLAG_FULL_DELTA = 8      /* the sampling weights as Eq. (delta_calc) states them: W_delta (and dW_delta) is
                                    [Hq, Hkv*d], one row per query head over ALL channels of the value row (the linear
                                    layer of the App. A listing), z[b,h,j] = sum_{h'} V[b,j,h',:] . W_delta[h, h'*d:(h'+1)*d].
                                    Without the flag W_delta is [Hq, d] and head h reads only its own KV head (the
                                    block-diagonal special case). Read by dma_mask_build, dma_mask_build_static,
                                    dma_delta_range, dma_mask_bwd, dma_mask_bwd_workspace and dma_step_host; needs
                                    roundup(Hq, d/8) * (Hkv*d + 64) * 4 <= 200 KiB */
};

typedef struct {
    int32_t B, Hq, Hkv, L, d;    /* d in {64, 128}; Hq % Hkv == 0; L >= 1 (query and key length are equal)      */
    int32_t w;                   /* keep window of Eq. (mask_combine), >= 1; values above L act as L            */
    int32_t causal;              /* 1: key j is visible to row i iff j <= i. 0 (non-causal, the App. A listing with an
                                    all-zero causal mask): every row sees every key, so all rows of a head keep the same
                                    min(w, L) keys; expiry[j] is then L for a kept key and 0 otherwise, key j is kept by the
                                    rows 0 <= i < expiry[j], and every bitmap row of a head is the same. bf16 (tensor-core kernels)
                                    always runs token-compacted in this mode (DMA_FLAG_COMPACT_KV is implied: the larger
                                    workspaces); dma_mask_build_varlen needs causal = 1              */
    int32_t dtype;               /* DMA_BF16 | DMA_FP32                                                         */
    int32_t tile_m, tile_n;      /* bitmap granularity (query rows x keys per bit); 0,0 = 128,128               */
    int32_t flags;               /* DMA_FLAG_*                                                                  */
    float softmax_scale;         /* 0 -> 1/sqrt(d)  (Alg. 1: S = Q K^T d^-1/2 + M)                              */
    int64_t q_stride[3];         /* batch, sequence, head strides of Q (also dQ) in elements; all 0 = contiguous*/
    int64_t k_stride[3];         /* same for K (also dK)                                                        */
    int64_t v_stride[3];         /* same for V (also dV)                                                        */
    int64_t o_stride[3];         /* same for O (also dO)                                                        */
} dma_problem_t;

/* Bytes of device workspace each stage needs for this problem (any pointer may be NULL to skip it).
 * Each workspace begins with a 256-byte header whose first int32 is the device status word. */
int dma_query_workspace(const dma_problem_t* p, size_t* mask_ws, size_t* fwd_ws, size_t* bwd_ws);

/* Number of uint32 words of the bitmap, [B, Hq, Tr, ceil(Tc/32)] with Tr = ceil(L/tile_m), Tc = ceil(L/tile_n). */
int dma_bitmap_words(const dma_problem_t* p, size_t* words);

/* Mask generation (Sec. 4.1).
 *   z[b,h,j]     = V[b,j,h/G,:] . W_delta[h,:]                        value projection, Eq. (delta_calc)
 *   bias[b,h,j]  = exp(A[h] * softplus(z))                             the dynamic weight delta; it is the additive
 *                                                                      mask value wherever the key is kept
 *   expiry[b,h,j]                                                      row i keeps key j iff j <= i < expiry[j]. This
 *        is the exact compact form of Eq. (mask_combine) read per query row over the causally visible keys:
 *        row i keeps the min(w, i+1) best keys under the order (delta descending, index ascending).
 *   bitmap       bit (kt % 32) of word [b,h,qt,kt/32] is 1 iff some (i in tile qt, j in tile kt) is kept: the
 *                block-level Judge test of Alg. 1 / Alg. 2.
 * delta is computed in fp32 in a fixed operation order so that its bit pattern, and therefore the selection,
 * is reproducible. W_delta is [Hq, d] fp32, A is [Hq] fp32. Supports both dtypes, d in {64,128}. */
int dma_mask_build(const dma_problem_t* p, const void* V, const float* W_delta, const float* A,
                   float* bias, int32_t* expiry, uint32_t* bitmap,
                   void* ws, size_t ws_bytes, void* cuda_stream);

/* Same computation and outputs as dma_mask_build, for callers that cannot supply a workspace. (The paper has no
 * counterpart: this is a property of the library, not of the method.) Some hosts forbid device allocation
 * at the point where the mask is built: an inference server that has handed all device memory to its own arena
 * and treats any later cudaMalloc as an error, or a plug-in that runs inside another framework's step and has no
 * allocator of its own to ask. This entry point allocates nothing and calls no allocating routine: its scratch is
 * a fixed 21 MiB array inside the library's device image, present on every GPU that loads the library until the
 * process exits.
 *   Limit: B * Hq * roundup(L, 256) <= 1,048,576 sort keys; beyond that it returns DMA_ERR_WORKSPACE and launches
 *   nothing (use dma_mask_build with a caller-provided workspace instead).
 *   The first call on each device looks up the array's device address (that device must be current, as for
 *   every call); make that first call before starting any stream capture. The address is remembered per device
 *   ordinal for the life of the process: it belongs to the device's primary context, so a process that calls
 *   cudaDeviceReset, or that runs this entry point under a context of its own (driver API) instead of the primary
 *   one, must not use it afterwards (use dma_mask_build there).
 *   All calls on a device share the one array. Nothing in it has to start at zero (each call rewrites what it
 *   reads), but two calls whose kernels overlap on the GPU, from different streams or threads, race on it:
 *   serialise them. */
int dma_mask_build_static(const dma_problem_t* p, const void* V, const float* W_delta, const float* A,
                          float* bias, int32_t* expiry, uint32_t* bitmap, void* cuda_stream);

/* Mask generation for sequences packed along the sequence axis (variable-length batches; the method applied to each
 * sequence on its own). cu_seqlens: DEVICE memory, nseq + 1 int32, cu[0] = 0 < cu[1] < ... < cu[nseq] = L: sequence s
 * owns positions cu[s] <= j < cu[s+1] of every batch entry. Row i sees the keys of its own sequence up to itself and
 * keeps the min(w, visible) best of them. Same outputs as dma_mask_build in packed coordinates: key j is kept by the
 * rows j <= i < expiry[j], and expiry[j] never passes the end of j's sequence, so no row reaches into another
 * sequence. dma_attn_fwd, dma_attn_bwd and dma_mask_bwd take the triple as it is: nothing else changes for packed
 * batches (the bitmap becomes block-diagonal, so whole key tiles of other sequences are skipped). The contents of
 * cu_seqlens are not checked (reading them would synchronise); offsets outside [0, L] are clamped. */
int dma_mask_build_varlen(const dma_problem_t* p, const void* V, const float* W_delta, const float* A,
                          const int32_t* cu_seqlens, int32_t nseq, float* bias, int32_t* expiry, uint32_t* bitmap,
                          void* ws, size_t ws_bytes, void* cuda_stream);

/* Forward (Sec. 4.2, Eq. (attention_output), Alg. 1): for each row i of head h
 *   s_j = q_i . k_j * scale + bias[j]   over keys with j <= i < expiry[j];   p = softmax(s);   O_i = sum p_j v_j
 *   lse_i = log sum_j exp(s_j)   (natural log; replaces Alg. 1's (l, m) pair)
 * Key tiles whose bitmap bit is 0 are neither loaded nor computed. Any self-consistent (bias, expiry, bitmap)
 * triple is accepted. bf16: tcgen05/TMA kernels, one instantiation for d = 128 and one for d = 64 (forward and backward);
 * fp32: CUDA-core kernel. */
int dma_attn_fwd(const dma_problem_t* p, const void* Q, const void* K, const void* V,
                 const float* bias, const int32_t* expiry, const uint32_t* bitmap,
                 void* O, float* lse, void* ws, size_t ws_bytes, void* cuda_stream);

/* Forward for a chunk of query rows (prefill in pieces over a KV cache; the same computation as dma_attn_fwd restricted
 * to the rows q_begin <= i < q_begin + q_len of the sequence of p->L keys, bottom-right aligned when q_begin + q_len = L):
 * Q and O are [B, q_len, Hq, d] (q_stride / o_stride, all 0 = packed with q_len rows), lse is [B, Hq, q_len]; K, V, bias
 * and expiry are those of the whole sequence (the mask built over all p->L keys). q_begin and q_len need no alignment.
 * bf16 (d = 128 or 64) runs the token-compacted kernel (its workspace size: dma_query_workspace with DMA_FLAG_COMPACT_KV set);
 * the other cases run the CUDA-core kernel. No bitmap is needed. */
int dma_attn_fwd_chunk(const dma_problem_t* p, int32_t q_begin, int32_t q_len, const void* Q, const void* K, const void* V,
                       const float* bias, const int32_t* expiry, void* O, float* lse, void* ws, size_t ws_bytes,
                       void* cuda_stream);

/* Backward (Sec. 4.3, Alg. 2, Eqs. (grad_v), (grad_s), (grad_m), (grad_qk)), mask and bias values held fixed:
 *   D_i = dO_i . O_i;  p_ij = exp(s_ij - lse_i);  dP_ij = dO_i . v_j;  dS_ij = p_ij (dP_ij - D_i)
 *   dV_j = sum_i p_ij dO_i;  dK_j = scale sum_i dS_ij q_i;  dQ_i = scale sum_j dS_ij k_j;  dM[b,h,j] = sum_i dS_ij
 * dK and dV are summed over the Hq/Hkv query heads that share a KV head; dM is per query head.
 * dQ is accumulated with floating-point atomics: its rounding depends on execution order. dK, dV (and O, lse of the
 * forward) are reproducible bit for bit from run to run on the tile path and the CUDA-core path; with
 * token-compacted execution dK and dV are accumulated with atomics too (one CTA per query head) and vary in the last
 * bits unless DMA_FLAG_DETERMINISTIC is set. */
int dma_attn_bwd(const dma_problem_t* p, const void* Q, const void* K, const void* V,
                 const void* O, const void* dO, const float* lse,
                 const float* bias, const int32_t* expiry, const uint32_t* bitmap,
                 void* dQ, void* dK, void* dV, float* dM,
                 void* ws, size_t ws_bytes, void* cuda_stream);

/* Mask-generation backward (Sec. 4.3: the bias gradient dM produced by dma_attn_bwd flows on to the sampling weights
 * and the gate; Eq. (delta_calc) differentiated with the top-w selection held fixed). With z = v_j . W_delta[h],
 * sp = softplus(z) and delta = exp(A[h] sp) = bias[b,h,j]:
 *   g = dM[b,h,j] delta;   dA[h] = sum_{b,j} g sp;   dz = g A[h] sigmoid(z);
 *   dW_delta[h,:] = sum_{b,j} dz v_j;      dV[b,j,h / (Hq/Hkv),:] += sum_{h in group} dz W_delta[h,:]
 * V, bias (the delta written by dma_mask_build), dM: inputs. dV [B,L,Hkv,d] (layout and strides of V, element type of
 * the problem) is IN/OUT: the contribution is added to what it holds (the attention backward's dV), in fp32, and
 * rounded once. dW_delta [Hq,d] and dA [Hq] fp32 are overwritten; their sums are formed in a fixed order (no
 * floating-point atomics). ws: dma_mask_bwd_workspace() bytes. All pointers device memory, 16-byte aligned. */
int dma_mask_bwd_workspace(const dma_problem_t* p, size_t* bytes);
int dma_mask_bwd(const dma_problem_t* p, const void* V, const float* W_delta, const float* A, const float* bias,
                 const float* dM, void* dV, float* dW_delta, float* dA, void* ws, size_t ws_bytes, void* cuda_stream);

/* Decoding (Sec. 3.2 for one query at the end of the sequence; Alg. 1 with the per-key mask M in R^N; the paper's
 * decode benchmark): p->L is the number N of cached keys, k_stride / v_stride describe the K / V caches
 * [B, >= N, Hkv, d] (a cache with spare capacity is a larger sequence stride), q and o are contiguous [B, Hq, d] in the
 * problem's element type, delta is the cache of dynamic weights [B, Hq, delta_ld] fp32 (delta_ld >= N entries per row).
 *
 * dma_delta_range: delta[b,h,j] = exp(A[h] softplus(V[b,j,h/G,:] . W_delta[h,:])) for the keys j in [j_begin, j_end)
 * only, with the same fixed fp32 arithmetic as dma_mask_build (bit-identical values): appends new keys to the cache.
 *
 * dma_decode: every (batch, query head) keeps the min(w, N) keys with the largest delta (ties to the lower index) and
 * returns o = softmax(q . K_sel^T scale + delta_sel) V_sel and its log-sum-exp lse [B, Hq] (natural log). sel_idx, if
 * not NULL, receives the kept key indices [B, Hq, min(w, N)] int32 in ascending order. Only the selected K and V rows
 * are read. ws: dma_decode_workspace() bytes. All pointers device memory, 16-byte aligned. */
int dma_delta_range(const dma_problem_t* p, const void* V, const float* W_delta, const float* A, float* delta, int64_t delta_ld,
                    int32_t j_begin, int32_t j_end, void* cuda_stream);
int dma_decode_workspace(const dma_problem_t* p, size_t* bytes);
int dma_decode(const dma_problem_t* p, const void* q, const void* K, const void* V, const float* delta, int64_t delta_ld,
               void* o, float* lse, int32_t* sel_idx, void* ws, size_t ws_bytes, void* cuda_stream);

/* Decoding with a carried state: one key is appended per step, so the set of the w best keys changes by at most one
 * member (the new key enters iff it beats the weakest kept key or the set is not full, and that weakest key leaves).
 * A step then costs O(w) whatever the number of cached keys: no scan of the delta row.
 *   state: device memory, dma_decode_state_bytes() bytes ([B, Hq] rows of 8 int32 of header (count, position and 64-bit
 *          order key of the weakest kept key) and p->w int32 kept key indices in no particular order), 16-byte aligned,
 *          owned by the caller; it depends on B, Hq and w only.
 *   dma_decode_state_init: the state for the first N = p->L cached keys (the selection of dma_decode).
 *   dma_decode_step: p->L = N counts the cached keys INCLUDING the key appended for this step (index N - 1), whose
 *          K, V and delta entries are already in the caches; `state` describes the first N - 1 keys on entry and all N
 *          on return. o, lse as dma_decode: the same keys are selected, so the results agree up to summation order.
 *          (N = 1 with a state whose count is 0, e.g. zero-filled memory, starts a sequence.)
 *   ws: dma_decode_workspace() bytes of the same problem. */
int dma_decode_state_bytes(const dma_problem_t* p, size_t* bytes);
int dma_decode_state_init(const dma_problem_t* p, const float* delta, int64_t delta_ld, void* state, void* ws, size_t ws_bytes,
                          void* cuda_stream);
int dma_decode_step(const dma_problem_t* p, const void* q, const void* K, const void* V, const float* delta, int64_t delta_ld,
                    void* state, void* o, float* lse, void* ws, size_t ws_bytes, void* cuda_stream);

/* The whole hot path on HOST buffers (all contiguous, default strides only): copies Q,K,V,(dO),W_delta,A into the
 * caller's device arena, runs dma_mask_build, dma_attn_fwd and, if `backward` != 0, dma_attn_bwd on the stream,
 * copies O, lse (and dQ,dK,dV,dM) back and synchronises the stream before returning. The copies run on two helper
 * streams that exist only for the duration of the call, so that they overlap the kernels; the step is cut into
 * independent (batch entry, group of KV heads) problems (up to four head groups, addressed inside the full tensors by
 * strides) so that the next group's inputs arrive and the previous group's results leave while a group computes; the
 * results are those of the device entry points on the same inputs. h* pointers are HOST memory
 * (pinned memory makes the copies asynchronous and faster); dev_arena is DEVICE memory, 256-byte aligned, of at
 * least dma_step_host_arena() bytes; hdO, hdQ, hdK, hdV, hdM may be NULL when `backward` is 0. */
int dma_step_host_arena(const dma_problem_t* p, int backward, size_t* bytes);
int dma_step_host(const dma_problem_t* p, int backward, const void* hQ, const void* hK, const void* hV, const void* hdO,
                  const float* hW_delta, const float* hA, void* hO, float* hlse, void* hdQ, void* hdK, void* hdV,
                  float* hdM, void* dev_arena, size_t arena_bytes, void* cuda_stream);

/* Synchronises the stream and returns the device status word of a workspace: 0, DMA_ERR_DEVICE_TIMEOUT or
 * DMA_ERR_MASK_OVERFLOW. */
int dma_read_status(const void* ws, void* cuda_stream);

/* Self-test of the bounded device-side waits (every mbarrier wait in the kernels gives up after a cycle limit, raises
 * the CTA's abort flag and leaves DMA_ERR_DEVICE_TIMEOUT in the workspace status word instead of hanging): launches
 * one small CTA that waits, with a ~2 ms limit, on a barrier nothing arrives at. Afterwards dma_read_status(ws) must
 * return DMA_ERR_DEVICE_TIMEOUT and the context stays usable. ws: any workspace of at least 256 bytes. */
int dma_selftest_wait_timeout(void* ws, size_t ws_bytes, void* cuda_stream);

/* Number of kernels the library has launched in this process (all entry points), for accounting. */
long long dma_launch_count(void);

/* Measurement hook (a property of the library; the paper has no counterpart). While recording is on, every dma_attn_fwd
 * and dma_attn_bwd call brackets its MAIN kernel (the attention kernel itself, not the small kernels before and after it:
 * key lists, D = rowsum(dO o O), accumulator conversion) with a pair of CUDA events on the caller's stream; up to 4096
 * pairs are kept, in call order. dma_kernel_timing(1) discards earlier records and starts recording, dma_kernel_timing(0)
 * stops. dma_kernel_timing_read waits for the recorded events and writes the elapsed milliseconds of each recorded
 * launch to ms[] and its stage to which[] (0 = forward, 1 = backward), at most `capacity` of them; *count receives the
 * number recorded. HOST pointers. Do not record while capturing a CUDA graph. */
int dma_kernel_timing(int enable);
int dma_kernel_timing_read(float* ms, int32_t* which, int32_t capacity, int32_t* count);

const char* dma_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* DMA_B200_H */
