/*
 * dapq.h - C ABI of the DapQ eviction scorer for NVIDIA B200 (sm_100a).
 *
 * DapQ (decoding-aligned KV cache compression via position-aware pseudo queries)
 * appends N synthetic tokens to a prompt of length L_p, gives them the positions
 * L_p .. L_p+N-1 of the first N decoding steps, and uses their queries as the
 * observation window that decides which prompt tokens stay in the KV cache.
 * This library is the step that runs after the extended prefill of one layer:
 *
 *   1. dapq_rope_pseudo_q  rotate the pseudo queries to their decode positions
 *                          (Section 4.1, "Positions(T_pseudo) = [L_p, ..., L_p+N-1]").
 *   2. dapq_score          S(j) = sum_i Attention(q_i, k_j)            (Section 4.2, Eq. 4)
 *                          with Attention = softmax(q K^T / sqrt(d_k)) (Appendix C, Theorem),
 *                          summed over the query heads of a GQA group.
 *   3. dapq_topk_select    M_retain = TopK_j S(j)                       (Section 4.2, Eq. 5)
 *   4. dapq_compact_kv     keep the K/V rows in M_retain, drop the rest and every
 *                          synthetic token (Section 4.2, last paragraph; Figure 1).
 *   5. dapq_evict          1-4 for one layer's cache on one stream (dapq_evict_layers: every layer;
 *                          dapq_evict_host, dapq_evict_layers_host: the same on host buffers).
 *   Also: dapq_recall (Section 3.3, Eq. 1-3), optional pooling of the scores before step 3.
 *
 * Conventions
 *   - One process drives one GPU.  All kernels are asynchronous on the caller's
 *     stream (a cudaStream_t passed as void*; NULL = the legacy default stream).
 *   - "device" pointers are caller-owned device memory that must stay valid until
 *     the stream work finishes; "host" pointers are read before the call returns.
 *   - The library allocates device memory only inside dapq_create (workspace sized
 *     from dapq_shape) and, on first use, inside dapq_evict_host / dapq_evict_layers_host
 *     (staging buffers, a copy stream, events).
 *   - Argument errors are returned synchronously and launch nothing.  A bounded
 *     device-side wait that gives up sets a status word that dapq_poll_status reads.
 *   - Outputs must not alias inputs.
 *
 * Layouts (d = head_dim = 128, G = n_q_heads / n_kv_heads, query head h reads KV head h / G)
 *   q_pre, q_rot  [B, H_q, N, d]   contiguous, element type = dapq_shape.dtype
 *   K, V cache    [H_kv, R, d]     strided view (strides in elements, d contiguous); the R rows
 *                                  are packed by sequence: sequence b owns rows
 *                                  cu_rows[b] .. cu_rows[b+1]-1 = L_b prompt rows followed by
 *                                  its N synthetic rows.  Keys are stored already rotated.
 *   scores        [H_kv, T]        fp32, T = sum_b L_b, sequence b at columns cu_prompt[b] ..
 *   idx           [H_kv, KT]       int32, KT = sum_b min(K_b, L_b); sequence-local prompt
 *                                  positions in [0, L_b), ascending within a sequence
 *   k_out, v_out  [H_kv, KT, d]    contiguous, same element type as the cache
 */
#ifndef DAPQ_H
#define DAPQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define DAPQ_API __attribute__((visibility("default")))
#else
#define DAPQ_API
#endif

typedef enum {
  DAPQ_OK = 0,
  DAPQ_ERR_INVALID_ARG = 1,   /* null pointer, non-positive size, inconsistent offsets */
  DAPQ_ERR_UNSUPPORTED = 2,   /* head_dim != 128, N > 128, misaligned strides, ... */
  DAPQ_ERR_WORKSPACE = 3,     /* call exceeds the sizes given to dapq_create */
  DAPQ_ERR_CUDA = 4,          /* a CUDA runtime / driver call failed (see dapq_last_error) */
  DAPQ_ERR_TIMEOUT = 5        /* a bounded device-side wait expired (dapq_poll_status) */
} dapq_status;

typedef enum { DAPQ_BF16 = 0, DAPQ_F32 = 1 } dapq_dtype;

enum { DAPQ_MAX_BATCH = 128, DAPQ_MAX_PSEUDO = 128, DAPQ_HEAD_DIM = 128, DAPQ_MAX_POOL_KERNEL = 127 };

/* Pooling of the accumulated scores before selection.  The paper specifies none for
 * DapQ (it mentions pooling only for the SnapKV / PyramidKV baselines), so NONE is the
 * default; MAX / AVG apply a 1-D window of odd width pool_kernel (3 .. DAPQ_MAX_POOL_KERNEL),
 * stride 1, clipped at the ends of each sequence (AVG is the mean of the positions that
 * exist).  With pooling on, dapq_topk_select and dapq_evict select on the pooled scores;
 * the scores that dapq_score and dapq_evict hand out are always the unpooled Eq. 4 sums. */
typedef enum { DAPQ_POOL_NONE = 0, DAPQ_POOL_MAX = 1, DAPQ_POOL_AVG = 2 } dapq_pool_mode;

/* dapq_shape.flags.  DAPQ_FLAG_CUDA_CORE_SCORER keeps the scorer on the CUDA-core kernels
 * (fp32 arithmetic on unrounded rotated queries) even where the tensor-core path applies.
 * DAPQ_FLAG_ROPE_INTERLEAVED: the rotation pairs channel 2c with 2c + 1 instead of c with
 * c + d/2 (Section 4.1 only says "RoPE"; the rotate-half pairing of the paper's Llama and Qwen
 * models is the default; the cache's keys must have been rotated with the same pairing).
 *
 * Precision of the rotated queries on the tensor-core path of dapq_evict (the paper states no
 * precision; Eq. 4 is evaluated with fp32 accumulation whatever the choice):
 *   default                 queries rounded to fp16 (11 significant bits), fp16 x fp16 MMAs, the bf16
 *                           keys converted to fp16 on the fly: exact for key magnitudes 2^-14 .. 65504,
 *                           larger keys saturate at 65504;
 *   DAPQ_FLAG_Q_BF16        queries rounded to bf16 (8 significant bits), bf16 x bf16 MMAs: any key
 *                           magnitude, the coarsest scores (caches with outlier channels can leave
 *                           the 2e-3 per-token band);
 *   DAPQ_FLAG_Q_LO_SWEEP1,  queries as a bf16 pair hi + lo (16 significant bits); the named sweep(s)
 *   DAPQ_FLAG_Q_LO_SWEEP2   (1 = row normalisers, 2 = column sums) add the lo part with a second MMA
 *                           pass: any key magnitude, the finest scores, twice the tensor work in
 *                           those sweeps.  Either flag implies bf16 queries. */
typedef enum {
  DAPQ_FLAG_CUDA_CORE_SCORER = 1, DAPQ_FLAG_ROPE_INTERLEAVED = 2, DAPQ_FLAG_Q_BF16 = 4, DAPQ_FLAG_Q_LO_SWEEP1 = 8,
  DAPQ_FLAG_Q_LO_SWEEP2 = 16
} dapq_flags;

typedef struct dapq_ctx dapq_ctx;

typedef struct {
  int32_t n_q_heads;        /* H_q                                               */
  int32_t n_kv_heads;       /* H_kv, divides H_q                                 */
  int32_t head_dim;         /* must be 128                                        */
  int32_t n_pseudo;         /* N, 1 .. 128                                        */
  int32_t max_batch;        /* largest B of any call, 1 .. DAPQ_MAX_BATCH         */
  int32_t dtype;            /* dapq_dtype of q, K and V                           */
  int64_t max_total_rows;   /* largest R = sum_b (L_b + N) of any call            */
  double  rope_base;        /* theta_c = rope_base^(-2c/d) unless inv_freq_host   */
  const double* inv_freq_host; /* host, optional [d/2] frequencies (scaled RoPE)  */
  float   softmax_scale;    /* 0 -> 1/sqrt(head_dim)                              */
  int32_t pool_mode;        /* dapq_pool_mode                                     */
  int32_t pool_kernel;      /* odd window width; ignored for DAPQ_POOL_NONE       */
  int32_t flags;            /* bit set of dapq_flags, normally 0                  */
} dapq_shape;

typedef struct {
  const void* k;                  /* device, [H_kv, R, d] view                    */
  const void* v;                  /* device, same geometry (may be NULL for dapq_score) */
  int64_t k_head_stride;          /* elements between KV heads                    */
  int64_t k_row_stride;           /* elements between rows (>= d, multiple of 8)  */
  int64_t v_head_stride;
  int64_t v_row_stride;
  const int32_t* cu_rows_host;    /* host [B+1], cu_rows[b+1]-cu_rows[b] = L_b + N */
  const int32_t* prompt_len_host; /* host [B], L_b >= 1                            */
  int32_t batch;                  /* B                                            */
  int32_t reserved;               /* must be 0                                    */
} dapq_cache_view;

/* Create a context on `device` (made current for the call).  Allocates the workspace.
 * Returns DAPQ_ERR_UNSUPPORTED for shapes outside the limits above. */
DAPQ_API dapq_status dapq_create(dapq_ctx** out, const dapq_shape* shape, int device);
DAPQ_API void dapq_destroy(dapq_ctx* ctx);

/* Text of the last error of this context (never NULL; valid until the next call).
 * With ctx == NULL: the reason the last dapq_create on this thread failed. */
DAPQ_API const char* dapq_last_error(const dapq_ctx* ctx);

/* Synchronises `stream`, then reads and clears the device status word.  Returns
 * DAPQ_ERR_TIMEOUT if any kernel since the last poll gave up on a bounded wait
 * (its results are then undefined), DAPQ_ERR_CUDA if the stream reports an error. */
DAPQ_API dapq_status dapq_poll_status(dapq_ctx* ctx, void* stream);

/* Number of kernels this context has launched so far (for benchmarks' accounting). */
DAPQ_API int64_t dapq_launch_count(const dapq_ctx* ctx);

/* Diagnostics (the paper has no counterpart): the bound, in SM clock cycles, on every device-side
 * wait of the tensor-core score kernels launched from now on; 0 restores the default (about one
 * second).  A wait that outlasts the bound makes its CTA raise the timeout status, see its copies and
 * MMAs in flight complete and return; dapq_poll_status then reports DAPQ_ERR_TIMEOUT and the
 * call's results are undefined.  A bound of a few cycles makes every kernel give up at once, which is
 * how the give-up path is tested. */
DAPQ_API dapq_status dapq_set_wait_limit(dapq_ctx* ctx, int64_t cycles);

/* Per-kernel timing for benchmarks (the paper has no counterpart).  While enabled, every
 * kernel launch is bracketed by CUDA events on its stream; dapq_profile(ctx, 1) also clears
 * the totals.  dapq_profile_read synchronises `stream` and returns, per kernel kind, the
 * summed device time in milliseconds and the number of launches since profiling was
 * enabled.  ms_out / count_out: host [DAPQ_PROF_KINDS], in the order of dapq_prof_kind. */
typedef enum {
  DAPQ_PROF_ROPE = 0, DAPQ_PROF_SWEEP1 = 1, DAPQ_PROF_LSE_MERGE = 2, DAPQ_PROF_SWEEP2 = 3,
  DAPQ_PROF_TOPK = 4, DAPQ_PROF_COMPACT = 5, DAPQ_PROF_POOL = 6, DAPQ_PROF_RECALL = 7, DAPQ_PROF_SLOT_SUM = 8,
  DAPQ_PROF_KINDS = 9
} dapq_prof_kind;
DAPQ_API dapq_status dapq_profile(dapq_ctx* ctx, int32_t enable);
DAPQ_API dapq_status dapq_profile_read(dapq_ctx* ctx, void* stream, double* ms_out, int64_t* count_out);

/* Frequency table of the Llama-3.1 long-context RoPE scaling, for dapq_shape.inv_freq_host (the
 * paper's efficiency runs, Appendix B.6, use Llama-3.1-8B-Instruct, whose keys are rotated with these
 * frequencies; Section 4.1 needs the pseudo queries rotated the same way).  Per channel pair c, with
 * theta_c = rope_base^(-2c/d) and wavelength 2 pi / theta_c: wavelengths below original_context /
 * high_freq_factor keep theta_c, those above original_context / low_freq_factor get theta_c / factor,
 * the band between is interpolated linearly in original_context / wavelength.  Llama-3.1 uses
 * rope_base 500000, factor 8, low 1, high 4, original_context 8192.
 * inv_freq_out: host [DAPQ_HEAD_DIM / 2].  Host arithmetic only; touches no device. */
DAPQ_API dapq_status dapq_rope_inv_freq_llama3(double rope_base, double factor, double low_freq_factor,
                                      double high_freq_factor, int32_t original_context, double* inv_freq_out);

/* Section 4.1: q_rot[b,h,i,:] = RoPE(q_pre[b,h,i,:], position pos_start[b] + i), rotate-half
 * pairing (channel c with c + d/2), angles formed in double precision.
 * q_pre, q_rot: device [B, H_q, N, d]; pos_start_host: host [B] (DapQ uses L_b; other
 * values give the paper's shifted-position ablation). */
DAPQ_API dapq_status dapq_rope_pseudo_q(dapq_ctx* ctx, const void* q_pre, const int32_t* pos_start_host,
                               int32_t batch, void* q_rot, void* stream);

/* Section 4.2, Eq. 4 with Attention = softmax(q K^T * scale) over the causal span of the
 * extended prefill: pseudo query i sees the L_b prompt keys and synthetic keys 0 .. i.
 *   scores[kvh, cu_prompt[b] + j] = sum_{g<G} sum_{i<N} P[b, kvh*G+g, i, j],  j < L_b.
 * q_rot: device (already rotated).  lse_in: device [B, H_q, N] natural-log sum-exp of each
 * pseudo query's visible logits, or NULL to have the library compute it (one extra sweep
 * over K).  lse_out (nullable): receives the log-sum-exp used.  syn_mass (nullable):
 * device [B, H_q], attention mass each head puts on the synthetic keys; for every KV head
 * sum_j scores + sum_g syn_mass = G * N. */
DAPQ_API dapq_status dapq_score(dapq_ctx* ctx, const void* q_rot, const dapq_cache_view* cache,
                       const float* lse_in, float* scores, float* lse_out, float* syn_mass,
                       void* stream);

/* Section 4.2, Eq. 5: for every (b, kvh) the min(K_b, L_b) positions with the largest
 * score; equal scores at the threshold go to the lower position; positions are written
 * in ascending order.  scores: device [H_kv, T] (finite, >= 0); cu_prompt_host: host
 * [B+1]; k_keep_host: host [B], K_b >= 1; idx_out: device [H_kv, KT].  If the context was
 * created with a pooling mode, the scores are pooled first (into the workspace). */
DAPQ_API dapq_status dapq_topk_select(dapq_ctx* ctx, const float* scores, const int32_t* cu_prompt_host,
                             const int32_t* k_keep_host, int32_t batch, int32_t* idx_out,
                             void* stream);

/* Section 4.2, pruning: k_out[kvh, cu_keep[b] + r, :] = K[kvh, cu_rows[b] + idx[kvh, cu_keep[b] + r], :]
 * and the same rows of V; a bit-exact copy.  Synthetic rows are never copied.
 * idx: device [H_kv, KT] as written by dapq_topk_select (entries outside [0, L_b) are
 * skipped and flagged through dapq_poll_status as DAPQ_ERR_INVALID_ARG). */
DAPQ_API dapq_status dapq_compact_kv(dapq_ctx* ctx, const dapq_cache_view* cache, const int32_t* idx,
                            const int32_t* k_keep_host, void* k_out, void* v_out, void* stream);

/* Section 3.3, Eq. 1-3: Recall_W = |M_gold ∩ M_pred| / |M_gold| per (sequence, KV head), for two
 * retained sets chosen with the same budgets on the same cache (e.g. a small observation window
 * against a large one).  idx_gold, idx_pred: device [H_kv, KT] as written by dapq_topk_select
 * (ascending within a sequence); recall_out: device [B, H_kv] fp32. */
DAPQ_API dapq_status dapq_recall(dapq_ctx* ctx, const int32_t* idx_gold, const int32_t* idx_pred,
                        const int32_t* prompt_len_host, const int32_t* k_keep_host, int32_t batch,
                        float* recall_out, void* stream);

/* Figure 1, the whole eviction step for one layer: rotate to positions L_b + i, score,
 * select, compact.  idx_out, scores_out may be NULL (kept in the workspace). */
DAPQ_API dapq_status dapq_evict(dapq_ctx* ctx, const void* q_pre, const dapq_cache_view* cache,
                       const int32_t* k_keep_host, void* k_out, void* v_out, int32_t* idx_out,
                       float* scores_out, void* stream);

/* dapq_evict for every layer of a model, in layer order on one stream, with a budget per layer
 * (Section 4.2 is applied to each layer's cache on its own; the paper keeps one budget for all
 * layers, the layer-wise budgets of the PyramidKV baseline in Section 5.1 are the general case).
 * q_pre, caches, k_out, v_out, idx_out: HOST arrays of n_layers entries holding what dapq_evict
 * takes for one layer (idx_out, or any entry of it, may be NULL).  k_keep_host: host
 * [n_layers, batch] when k_keep_layer_stride = batch, or one row shared by all layers when
 * k_keep_layer_stride = 0.  Every layer uses the same workspace, so the layers run back to back;
 * only launches are issued (no copies, no synchronisation), which makes the whole call
 * capturable into a CUDA graph.  Stops at the first layer that fails and returns its status. */
DAPQ_API dapq_status dapq_evict_layers(dapq_ctx* ctx, int32_t n_layers, const void* const* q_pre,
                              const dapq_cache_view* caches, const int32_t* k_keep_host,
                              int64_t k_keep_layer_stride, void* const* k_out, void* const* v_out,
                              int32_t* const* idx_out, void* stream);

/* dapq_evict for callers whose tensors live in host memory: q_pre, the cache view's k / v
 * and k_out / v_out / idx_out are HOST pointers (pinned memory gives full copy speed).
 * Copies q_pre and K to device staging buffers owned by the context (allocated on first
 * use, sized from dapq_shape), runs dapq_evict, copies the results back and synchronises
 * `stream` before returning.  Of V only the retained rows are needed: when the caller's V is
 * page-locked memory that the device can address (cudaHostAlloc, cudaHostRegister), the
 * compaction kernel reads those rows from it directly and V is never copied as a whole;
 * pageable V is staged like K. */
DAPQ_API dapq_status dapq_evict_host(dapq_ctx* ctx, const void* q_pre_host, const dapq_cache_view* cache_host,
                            const int32_t* k_keep_host, void* k_out_host, void* v_out_host,
                            int32_t* idx_out_host, void* stream);

/* dapq_evict_host for every layer of a model (arguments as in dapq_evict_layers, all data
 * pointers HOST pointers).  Two staging sets and a copy stream owned by the context let the
 * host-to-device copies of layer l + 1 run beside the kernels and the device-to-host copies of
 * layer l; the call returns after `stream` has been synchronised.  Not capturable into a graph. */
DAPQ_API dapq_status dapq_evict_layers_host(dapq_ctx* ctx, int32_t n_layers, const void* const* q_pre_host,
                                   const dapq_cache_view* caches_host, const int32_t* k_keep_host,
                                   int64_t k_keep_layer_stride, void* const* k_out_host,
                                   void* const* v_out_host, int32_t* const* idx_out_host, void* stream);

/* The paper has no counterpart to this entry point; it exists for callers that may not
 * allocate device memory at the point where they need scores: engines whose own allocator owns
 * the whole device, plug-ins running after a "no more driver allocations" point, code between a
 * memory-pool snapshot and its restore.  dapq_create allocates a workspace, so such callers
 * cannot build a context; this call needs none and calls no cudaMalloc / cudaFree or any
 * allocating library routine.
 *
 * It computes what dapq_score computes (Eq. 4 scores per KV head, fp32 arithmetic on the CUDA
 * cores, both sweeps) from shape fields only: n_q_heads, n_kv_heads, head_dim, n_pseudo, dtype
 * and softmax_scale of `shape` are read, the rest is ignored.  q_rot (device, already rotated,
 * element type shape->dtype), cache->k (device) and scores (device, [H_kv, T]) are the caller's;
 * cache->v is not read.
 *
 * The scratch of the two sweeps lives in one fixed array of DAPQ_STATIC_SCRATCH_BYTES inside
 * the library image, which every GPU that loads the library holds until the process exits.  A
 * call needs  round_up(B * H_q * N * 4, 256)  +  sum_b (ceil(L_b / 512) + 1) * H_q * N * 8  bytes of
 * it (at H_q = 32, N = 64 a single prompt of up to 64512 tokens fits: 8192 + 127 * 16384 bytes); a
 * larger call returns DAPQ_ERR_WORKSPACE and launches nothing.  All calls on a device share the
 * array: calls whose kernels can overlap on the GPU (different streams, no dependency) race on
 * it and must be ordered by the caller.  Nothing in it needs clearing between calls.
 *
 * The FIRST call on each device is a warm-up and is not allocation-free: with that device current
 * it resolves the array's device address, which makes the CUDA runtime load the module that holds
 * the array, and it touches every kernel this entry point can launch so that their code is brought
 * to the device then and not by some later call (the runtime loads a kernel's code at its first
 * use, and that takes device memory).  Make that first call (any valid small problem will do)
 * before the point from which the process may no longer allocate, and outside any stream capture.
 * Every later call on that device, whatever its shape or dtype, allocates nothing.
 * err_out (nullable, host): receives a NUL-terminated reason when the status is not DAPQ_OK. */
enum { DAPQ_STATIC_SCRATCH_BYTES = 2 * 1024 * 1024 };
DAPQ_API dapq_status dapq_score_static(const dapq_shape* shape, int device, const void* q_rot,
                              const dapq_cache_view* cache, float* scores, void* stream,
                              char* err_out, size_t err_len);

#ifdef __cplusplus
}
#endif
#endif /* DAPQ_H */
