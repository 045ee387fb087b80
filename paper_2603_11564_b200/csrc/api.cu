// C ABI of libdapq: context, argument checking, workspace, and the launch sequences.
// See include/dapq.h for the contract of every entry point.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <new>
#include <vector>

#include "dapq_internal.cuh"

using namespace dapq;

struct dapq_ctx {
  int device = 0;
  dapq_shape shape{};
  Dims dims{};
  int elem_bytes = 2;
  int n_sm = 148;
  int64_t max_chunks = 0;
  int64_t q_rows_max = 0;        // max_batch * H_q * N
  // device workspace
  double* inv_freq = nullptr;    // [d/2]
  int* status = nullptr;         // device status word
  void* q_rot = nullptr;         // [max_batch, H_q, N, d]
  float2* part = nullptr;        // [max_chunks, H_q, N]
  float* lse2 = nullptr;         // [max_batch, H_q, N]
  float* scores = nullptr;       // [H_kv, max_total_rows]
  float* pooled = nullptr;       // [H_kv, max_total_rows] (pooling only)
  float* slots = nullptr;        // [query groups, H_kv, max_total_rows] (sized for groups of 256 query rows; used when sweep 2 has more than one group)
  long long wait_limit = 0;      // cycles a device-side wait may take (0: the default, about a second)
  int32_t* idx = nullptr;        // [H_kv, max_total_rows]
  // staging for the host-buffer entry points (allocated on first use): two sets, so that the copies of one
  // layer run beside the kernels of the layer before
  struct HostStage {
    void *q = nullptr, *k = nullptr, *v = nullptr, *ko = nullptr, *vo = nullptr;
    int32_t* idx = nullptr;
    cudaEvent_t in_done = nullptr;    // the layer's inputs have arrived (recorded on the copy stream)
    cudaEvent_t out_done = nullptr;   // the layer's results have left (recorded on the caller's stream)
  } hs[2];
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t fork = nullptr;         // orders the copy stream behind what the caller's stream already holds
  LaunchLog log;
  char err[512] = "";
};

// ---- launch accounting and per-kernel event timing ----------------------------------------
namespace dapq {
struct ProfImpl {
  std::vector<cudaEvent_t> pool;      // event pairs, reused after every drain
  std::vector<int> kinds;             // kind of each pending pair
  double ms[kKindCount] = {};
  int64_t count[kKindCount] = {};
  ~ProfImpl() { for (cudaEvent_t e : pool) cudaEventDestroy(e); }
};

void LaunchLog::begin(int kind, cudaStream_t s) {
  ++n_launch;
  if (!profiling) return;
  ProfImpl* p = static_cast<ProfImpl*>(impl);
  const size_t n = p->kinds.size();
  while (p->pool.size() < 2 * (n + 1)) {
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) { profiling = false; return; }
    p->pool.push_back(e);
  }
  p->kinds.push_back(kind);
  cudaEventRecord(p->pool[2 * n], s);
}

void LaunchLog::end(cudaStream_t s) {
  if (!profiling) return;
  ProfImpl* p = static_cast<ProfImpl*>(impl);
  cudaEventRecord(p->pool[2 * (p->kinds.size() - 1) + 1], s);
}
}  // namespace dapq

namespace {

// Message of the last failed dapq_create on this thread (there is no context to hold it).
thread_local char g_create_err[256] = "";

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

dapq_status fail(dapq_ctx* ctx, dapq_status st, const char* fmt, ...) {
  if (ctx) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
    va_end(ap);
  }
  return st;
}

dapq_status cuda_fail(dapq_ctx* ctx, cudaError_t e, const char* what) {
  return fail(ctx, DAPQ_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define DAPQ_CUDA(ctx, call)                                        \
  do {                                                              \
    cudaError_t e_ = (call);                                        \
    if (e_ != cudaSuccess) return cuda_fail((ctx), e_, #call);      \
  } while (0)

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Fill the sequence table from the caller's host arrays and check it against the context.
// Any of cu_rows / prompt_len may come from a cache view; k_keep and pos_start are optional.
dapq_status build_table(dapq_ctx* ctx, int32_t batch, const int32_t* cu_rows, const int32_t* prompt_len,
                        const int32_t* cu_prompt, const int32_t* k_keep, const int32_t* pos_start,
                        SeqTable* t) {
  const dapq_shape& sh = ctx->shape;
  if (batch < 1) return fail(ctx, DAPQ_ERR_INVALID_ARG, "batch must be >= 1 (got %d)", batch);
  if (batch > sh.max_batch)
    return fail(ctx, DAPQ_ERR_WORKSPACE, "batch %d exceeds max_batch %d", batch, sh.max_batch);
  memset(t, 0, sizeof(*t));
  t->batch = batch;
  int64_t rows = 0, prompt = 0, keep = 0, chunks = 0;
  for (int b = 0; b < batch; ++b) {
    int64_t L;
    if (prompt_len) {
      L = prompt_len[b];
    } else if (cu_prompt) {
      L = (int64_t)cu_prompt[b + 1] - cu_prompt[b];
    } else {
      L = 1;  // rope-only tables carry no lengths
    }
    if (L < 1) return fail(ctx, DAPQ_ERR_INVALID_ARG, "prompt length of sequence %d is %lld (must be >= 1)", b, (long long)L);
    if (cu_prompt && cu_prompt[b] != prompt)
      return fail(ctx, DAPQ_ERR_INVALID_ARG, "cu_prompt[%d] = %d, expected %lld", b, cu_prompt[b], (long long)prompt);
    if (cu_rows) {
      if (b == 0 && cu_rows[0] < 0) return fail(ctx, DAPQ_ERR_INVALID_ARG, "cu_rows[0] is negative");
      if ((int64_t)cu_rows[b + 1] - cu_rows[b] != L + sh.n_pseudo)
        return fail(ctx, DAPQ_ERR_INVALID_ARG,
                    "sequence %d owns %lld cache rows, expected L_b + N = %lld", b,
                    (long long)((int64_t)cu_rows[b + 1] - cu_rows[b]), (long long)(L + sh.n_pseudo));
      t->cu_rows[b] = cu_rows[b];
      t->cu_rows[b + 1] = cu_rows[b + 1];
    } else {
      t->cu_rows[b] = (int32_t)rows;
      t->cu_rows[b + 1] = (int32_t)(rows + L + sh.n_pseudo);
    }
    int64_t kb = L;
    if (k_keep) {
      if (k_keep[b] < 1) return fail(ctx, DAPQ_ERR_INVALID_ARG, "k_keep[%d] = %d (must be >= 1)", b, k_keep[b]);
      kb = k_keep[b] < L ? k_keep[b] : L;
    }
    t->prompt_len[b] = (int32_t)L;
    t->pos_start[b] = pos_start ? pos_start[b] : (int32_t)L;
    if (pos_start && pos_start[b] < 0) return fail(ctx, DAPQ_ERR_INVALID_ARG, "pos_start[%d] is negative", b);
    t->cu_prompt[b] = (int32_t)prompt;
    t->cu_keep[b] = (int32_t)keep;
    rows += L + sh.n_pseudo;
    prompt += L;
    keep += kb;
    chunks += (L + kChunkKeys - 1) / kChunkKeys + 1;
  }
  t->cu_prompt[batch] = (int32_t)prompt;
  t->cu_keep[batch] = (int32_t)keep;
  const int64_t last_row = cu_rows ? cu_rows[batch] : rows;
  if ((prompt_len || cu_prompt) && last_row > sh.max_total_rows)
    return fail(ctx, DAPQ_ERR_WORKSPACE, "%lld cache rows exceed max_total_rows %lld",
                (long long)last_row, (long long)sh.max_total_rows);
  if ((prompt_len || cu_prompt) && chunks > ctx->max_chunks)
    return fail(ctx, DAPQ_ERR_WORKSPACE, "%lld work chunks of %d keys exceed the %lld the workspace was sized for "
                "(more or longer sequences than max_batch / max_total_rows allow)",
                (long long)chunks, kChunkKeys, (long long)ctx->max_chunks);
  return DAPQ_OK;
}

dapq_status check_view(dapq_ctx* ctx, const dapq_cache_view* cv, bool need_v, bool host, CacheDev* out) {
  if (!cv) return fail(ctx, DAPQ_ERR_INVALID_ARG, "cache view is NULL");
  if (!cv->k || (need_v && !cv->v)) return fail(ctx, DAPQ_ERR_INVALID_ARG, "cache view has a NULL K or V pointer");
  if (!cv->cu_rows_host || !cv->prompt_len_host)
    return fail(ctx, DAPQ_ERR_INVALID_ARG, "cache view needs cu_rows_host and prompt_len_host");
  if (cv->reserved != 0) return fail(ctx, DAPQ_ERR_INVALID_ARG, "cache view reserved field must be 0");
  const int per16 = 16 / ctx->elem_bytes;
  const bool use_v = cv->v != nullptr;
  if (cv->k_row_stride < kHeadDim || cv->k_head_stride < 0 || (use_v && (cv->v_row_stride < kHeadDim || cv->v_head_stride < 0)))
    return fail(ctx, DAPQ_ERR_INVALID_ARG, "row strides must be >= head_dim and head strides >= 0");
  if (!host) {
    if (cv->k_row_stride % per16 || cv->k_head_stride % per16 || !aligned16(cv->k) ||
        (use_v && (cv->v_row_stride % per16 || cv->v_head_stride % per16 || !aligned16(cv->v))))
      return fail(ctx, DAPQ_ERR_UNSUPPORTED, "K/V base pointers and strides must be multiples of 16 bytes");
  }
  out->k = cv->k;
  out->v = cv->v;
  out->k_head_stride = cv->k_head_stride;
  out->k_row_stride = cv->k_row_stride;
  out->v_head_stride = cv->v_head_stride;
  out->v_row_stride = cv->v_row_stride;
  return DAPQ_OK;
}

// The tensor-core scorer takes bf16 caches whose query block is at least half an MMA tile high;
// everything else (fp32 storage, tiny windows, views TMA cannot describe, syn_mass requests)
// goes to the CUDA-core scorer.
bool wants_umma(const dapq_ctx* ctx) {
  return ctx->shape.dtype == DAPQ_BF16 && !(ctx->shape.flags & DAPQ_FLAG_CUDA_CORE_SCORER) &&
         ctx->dims.group * ctx->dims.n_pseudo >= 64;
}

dapq_status run_score_umma(dapq_ctx* ctx, const UmmaPlan& plan, const SeqTable& t, const float* lse_in,
                           float* scores, int64_t score_stride, float* lse_out, cudaStream_t s) {
  cudaError_t e = launch_score_umma(plan, t, ctx->dims, lse_in, ctx->part, scores, score_stride,
                                    lse_out, ctx->status, ctx->wait_limit, s, &ctx->log);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "tensor-core score kernels (two-part bf16 queries)");
  return DAPQ_OK;
}

dapq_status run_score_qg(dapq_ctx* ctx, const QgPlan& plan, const SeqTable& t, const float* lse_in,
                         float* scores, int64_t score_stride, float* lse_out, bool after_rope, cudaStream_t s) {
  cudaError_t e = launch_score_qg(plan, t, ctx->dims, lse_in, ctx->part, ctx->slots, scores, score_stride, lse_out,
                                  ctx->lse2, ctx->status, ctx->wait_limit, after_rope, s, &ctx->log);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "tensor-core score kernels");
  return DAPQ_OK;
}

// The older tensor-core kernels (a second MMA pass with the low-order bf16 part of the queries) serve
// the contexts that ask for that part in either sweep.
bool wants_lo(const dapq_ctx* ctx) { return (ctx->shape.flags & (DAPQ_FLAG_Q_LO_SWEEP1 | DAPQ_FLAG_Q_LO_SWEEP2)) != 0; }

dapq_status run_score(dapq_ctx* ctx, int q_dtype, const void* q_rot, const CacheDev& cd, const SeqTable& t,
                      const float* lse_in, float* scores, int64_t score_stride, float* lse_out,
                      float* syn_mass, cudaStream_t s) {
  cudaError_t e = launch_score_fma(ctx->shape.dtype, q_dtype, q_rot, cd, t, ctx->dims, lse_in, ctx->part, ctx->max_chunks, ctx->n_sm,
                                   ctx->lse2, scores, score_stride, lse_out, syn_mass, s, &ctx->log);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "score kernels");
  return DAPQ_OK;
}

// Eq. 5 on the scores, or on their pooled image if the context asks for pooling.
dapq_status run_select(dapq_ctx* ctx, const float* scores, int64_t score_stride, int32_t* idx, int64_t idx_stride,
                       const SeqTable& t, cudaStream_t s) {
  cudaError_t e;
  if (ctx->shape.pool_mode != DAPQ_POOL_NONE) {
    e = launch_pool(scores, ctx->pooled, score_stride, t, ctx->dims.n_kv_heads, ctx->shape.pool_kernel,
                    ctx->shape.pool_mode, s, &ctx->log);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "pooling kernel");
    scores = ctx->pooled;
  }
  e = launch_topk(scores, score_stride, idx, idx_stride, t, ctx->dims.n_kv_heads, s, &ctx->log);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "top-k kernel");
  return DAPQ_OK;
}

}  // namespace

extern "C" {

dapq_status dapq_create(dapq_ctx** out, const dapq_shape* sh, int device) {
  if (!out || !sh) return DAPQ_ERR_INVALID_ARG;
  *out = nullptr;
  dapq_ctx* ctx = new (std::nothrow) dapq_ctx();
  if (!ctx) return DAPQ_ERR_CUDA;
  // Errors before the context exists are reported through a context that is then freed:
  // keep the message reachable by returning the status only.
  auto bail = [&](dapq_status st, const char* why) {
    snprintf(g_create_err, sizeof(g_create_err), "dapq_create: %s", why);
    dapq_destroy(ctx);
    return st;
  };
  if (sh->head_dim != kHeadDim) return bail(DAPQ_ERR_UNSUPPORTED, "head_dim must be 128");
  if (sh->n_pseudo < 1 || sh->n_pseudo > kMaxPseudo) return bail(DAPQ_ERR_UNSUPPORTED, "n_pseudo must be in 1..128");
  if (sh->n_q_heads < 1 || sh->n_kv_heads < 1 || sh->n_q_heads % sh->n_kv_heads)
    return bail(DAPQ_ERR_INVALID_ARG, "n_kv_heads must divide n_q_heads");
  if (sh->max_batch < 1 || sh->max_total_rows < 1) return bail(DAPQ_ERR_INVALID_ARG, "max_batch and max_total_rows must be >= 1");
  if (sh->max_batch > kMaxBatch || sh->max_total_rows > 0x7fffffffLL)
    return bail(DAPQ_ERR_UNSUPPORTED, "max_batch > 128 or max_total_rows >= 2^31");
  if (sh->dtype != DAPQ_BF16 && sh->dtype != DAPQ_F32) return bail(DAPQ_ERR_INVALID_ARG, "unknown dtype");
  if (sh->flags & ~(DAPQ_FLAG_CUDA_CORE_SCORER | DAPQ_FLAG_ROPE_INTERLEAVED | DAPQ_FLAG_Q_BF16 | DAPQ_FLAG_Q_LO_SWEEP1 |
                    DAPQ_FLAG_Q_LO_SWEEP2))
    return bail(DAPQ_ERR_INVALID_ARG, "unknown flag");
  if (sh->pool_mode != DAPQ_POOL_NONE && sh->pool_mode != DAPQ_POOL_MAX && sh->pool_mode != DAPQ_POOL_AVG)
    return bail(DAPQ_ERR_INVALID_ARG, "unknown pool_mode");
  if (sh->pool_mode != DAPQ_POOL_NONE && (sh->pool_kernel < 3 || sh->pool_kernel > DAPQ_MAX_POOL_KERNEL || sh->pool_kernel % 2 == 0))
    return bail(DAPQ_ERR_UNSUPPORTED, "pool_kernel must be odd, 3 .. 127");
  if (!sh->inv_freq_host && !(sh->rope_base > 0.0)) return bail(DAPQ_ERR_INVALID_ARG, "rope_base must be > 0");
  if (!(sh->softmax_scale >= 0.f)) return bail(DAPQ_ERR_INVALID_ARG, "softmax_scale must be >= 0");

  ctx->device = device;
  ctx->shape = *sh;
  ctx->shape.inv_freq_host = nullptr;
  ctx->elem_bytes = sh->dtype == DAPQ_BF16 ? 2 : 4;
  ctx->dims.n_q_heads = sh->n_q_heads;
  ctx->dims.n_kv_heads = sh->n_kv_heads;
  ctx->dims.group = sh->n_q_heads / sh->n_kv_heads;
  ctx->dims.n_pseudo = sh->n_pseudo;
  ctx->dims.rope_interleaved = (sh->flags & DAPQ_FLAG_ROPE_INTERLEAVED) ? 1 : 0;
  const double scale = sh->softmax_scale > 0.f ? (double)sh->softmax_scale : 1.0 / sqrt((double)kHeadDim);
  ctx->dims.scale_log2e = (float)(scale * 1.4426950408889634074);

  DeviceGuard guard(device);
  if (!guard.ok) return bail(DAPQ_ERR_CUDA, "cannot make the device current");
  double freq[kHeadDim / 2];
  for (int c = 0; c < kHeadDim / 2; ++c)
    freq[c] = sh->inv_freq_host ? sh->inv_freq_host[c] : pow(sh->rope_base, -2.0 * c / (double)kHeadDim);
  if (cudaDeviceGetAttribute(&ctx->n_sm, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || ctx->n_sm < 1)
    return bail(DAPQ_ERR_CUDA, "cannot query the device");
  // partials of the CUDA-core sweeps: the chunks at 512 keys each, plus room to cut small inputs
  // finer (down to 64 keys) until every SM has two CTAs
  ctx->max_chunks = (sh->max_total_rows + kChunkKeys - 1) / kChunkKeys + 2LL * sh->max_batch +
                    (2LL * ctx->n_sm + sh->n_kv_heads - 1) / sh->n_kv_heads;
  const size_t hq_n = (size_t)sh->n_q_heads * sh->n_pseudo;
  ctx->q_rows_max = (int64_t)sh->max_batch * hq_n;
  size_t part_elems = (size_t)ctx->max_chunks * hq_n;
  const size_t part_umma = (size_t)umma_part_elems(sh->max_batch, sh->n_q_heads, sh->n_kv_heads, sh->n_pseudo);
  if (part_umma > part_elems) part_elems = part_umma;
  const size_t rows = (size_t)sh->max_total_rows;
  bool ok = true;
  ok = ok && cudaMalloc(&ctx->inv_freq, sizeof(freq)) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->status, sizeof(int)) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->q_rot, (size_t)sh->max_batch * hq_n * kHeadDim * sizeof(float)) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->part, part_elems * sizeof(float2)) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->lse2, ((size_t)sh->max_batch * hq_n + 32) * sizeof(float)) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->scores, (size_t)sh->n_kv_heads * rows * sizeof(float)) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->idx, (size_t)sh->n_kv_heads * rows * sizeof(int32_t)) == cudaSuccess;
  if (sh->pool_mode != DAPQ_POOL_NONE)
    ok = ok && cudaMalloc(&ctx->pooled, (size_t)sh->n_kv_heads * rows * sizeof(float)) == cudaSuccess;
  if (sh->dtype == DAPQ_BF16 && qg_groups(ctx->dims) > 1)
    ok = ok && cudaMalloc(&ctx->slots, (size_t)qg_groups(ctx->dims) * sh->n_kv_heads * rows * sizeof(float)) == cudaSuccess;
  ok = ok && cudaMemcpy(ctx->inv_freq, freq, sizeof(freq), cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemset(ctx->status, 0, sizeof(int)) == cudaSuccess;
  if (!ok) { cudaGetLastError(); return bail(DAPQ_ERR_CUDA, "workspace allocation failed"); }
  *out = ctx;
  return DAPQ_OK;
}

void dapq_destroy(dapq_ctx* ctx) {
  if (!ctx) return;
  {
    DeviceGuard guard(ctx->device);
    void* bufs[] = {ctx->inv_freq, ctx->status, ctx->q_rot, ctx->part, ctx->lse2, ctx->scores, ctx->pooled, ctx->slots, ctx->idx};
    for (void* p : bufs)
      if (p) cudaFree(p);
    for (auto& st : ctx->hs) {
      void* sb[] = {st.q, st.k, st.v, st.ko, st.vo, st.idx};
      for (void* p : sb)
        if (p) cudaFree(p);
      if (st.in_done) cudaEventDestroy(st.in_done);
      if (st.out_done) cudaEventDestroy(st.out_done);
    }
    if (ctx->fork) cudaEventDestroy(ctx->fork);
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  }
  delete static_cast<dapq::ProfImpl*>(ctx->log.impl);
  delete ctx;
}

const char* dapq_last_error(const dapq_ctx* ctx) { return ctx ? ctx->err : g_create_err; }

int64_t dapq_launch_count(const dapq_ctx* ctx) { return ctx ? ctx->log.n_launch : 0; }

dapq_status dapq_rope_inv_freq_llama3(double rope_base, double factor, double low_freq_factor, double high_freq_factor,
                                      int32_t original_context, double* inv_freq_out) {
  if (!inv_freq_out || !(rope_base > 0.0) || !(factor >= 1.0) || !(low_freq_factor > 0.0) ||
      !(high_freq_factor > low_freq_factor) || original_context < 1)
    return DAPQ_ERR_INVALID_ARG;
  const double two_pi = 6.283185307179586476925286766559;
  const double short_wave = original_context / high_freq_factor, long_wave = original_context / low_freq_factor;
  for (int c = 0; c < kHeadDim / 2; ++c) {
    const double f = pow(rope_base, -2.0 * c / (double)kHeadDim), wave = two_pi / f;
    double g = f;
    if (wave > long_wave) {
      g = f / factor;
    } else if (wave >= short_wave) {
      const double smooth = (original_context / wave - low_freq_factor) / (high_freq_factor - low_freq_factor);
      g = (1.0 - smooth) * f / factor + smooth * f;
    }
    inv_freq_out[c] = g;
  }
  return DAPQ_OK;
}

dapq_status dapq_set_wait_limit(dapq_ctx* ctx, int64_t cycles) {
  if (!ctx) return DAPQ_ERR_INVALID_ARG;
  if (cycles < 0) return fail(ctx, DAPQ_ERR_INVALID_ARG, "dapq_set_wait_limit: negative limit");
  ctx->wait_limit = cycles;
  return DAPQ_OK;
}

dapq_status dapq_poll_status(dapq_ctx* ctx, void* stream) {
  if (!ctx) return DAPQ_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  cudaStream_t s = (cudaStream_t)stream;
  int word = 0;
  DAPQ_CUDA(ctx, cudaStreamSynchronize(s));
  DAPQ_CUDA(ctx, cudaMemcpy(&word, ctx->status, sizeof(int), cudaMemcpyDeviceToHost));
  if (word) DAPQ_CUDA(ctx, cudaMemset(ctx->status, 0, sizeof(int)));
  if (word & kStatusTimeout) return fail(ctx, DAPQ_ERR_TIMEOUT, "a kernel gave up on a bounded wait; its results are undefined");
  if (word & kStatusBadIndex) return fail(ctx, DAPQ_ERR_INVALID_ARG, "dapq_compact_kv skipped indices outside [0, L_b)");
  if (word & kStatusSmemAlign)
    return fail(ctx, DAPQ_ERR_UNSUPPORTED, "the score kernels found their shared memory off a 1024-byte boundary and did nothing");
  return DAPQ_OK;
}

dapq_status dapq_profile(dapq_ctx* ctx, int32_t enable) {
  if (!ctx) return DAPQ_ERR_INVALID_ARG;
  if (!ctx->log.impl) {
    ctx->log.impl = new (std::nothrow) dapq::ProfImpl();
    if (!ctx->log.impl) return fail(ctx, DAPQ_ERR_CUDA, "out of host memory");
  }
  dapq::ProfImpl* p = static_cast<dapq::ProfImpl*>(ctx->log.impl);
  if (enable) {
    p->kinds.clear();
    for (int k = 0; k < kKindCount; ++k) { p->ms[k] = 0.0; p->count[k] = 0; }
  }
  ctx->log.profiling = enable != 0;
  return DAPQ_OK;
}

dapq_status dapq_profile_read(dapq_ctx* ctx, void* stream, double* ms_out, int64_t* count_out) {
  if (!ctx || !ms_out || !count_out) return DAPQ_ERR_INVALID_ARG;
  dapq::ProfImpl* p = static_cast<dapq::ProfImpl*>(ctx->log.impl);
  if (!p) return fail(ctx, DAPQ_ERR_INVALID_ARG, "profiling was never enabled");
  DeviceGuard guard(ctx->device);
  DAPQ_CUDA(ctx, cudaStreamSynchronize((cudaStream_t)stream));
  for (size_t i = 0; i < p->kinds.size(); ++i) {
    float ms = 0.f;
    DAPQ_CUDA(ctx, cudaEventElapsedTime(&ms, p->pool[2 * i], p->pool[2 * i + 1]));
    p->ms[p->kinds[i]] += ms;
    p->count[p->kinds[i]] += 1;
  }
  p->kinds.clear();
  for (int k = 0; k < kKindCount; ++k) { ms_out[k] = p->ms[k]; count_out[k] = p->count[k]; }
  return DAPQ_OK;
}

dapq_status dapq_rope_pseudo_q(dapq_ctx* ctx, const void* q_pre, const int32_t* pos_start_host,
                               int32_t batch, void* q_rot, void* stream) {
  if (!ctx) return DAPQ_ERR_INVALID_ARG;
  if (!q_pre || !q_rot || !pos_start_host) return fail(ctx, DAPQ_ERR_INVALID_ARG, "dapq_rope_pseudo_q: NULL argument");
  SeqTable t;
  dapq_status st = build_table(ctx, batch, nullptr, nullptr, nullptr, nullptr, pos_start_host, &t);
  if (st != DAPQ_OK) return st;
  DeviceGuard guard(ctx->device);
  cudaError_t e = launch_rope(ctx->shape.dtype, ctx->shape.dtype, 0, q_pre, q_rot, ctx->inv_freq, t, ctx->dims, false, (cudaStream_t)stream,
                              &ctx->log);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "rope kernel");
  return DAPQ_OK;
}

dapq_status dapq_score(dapq_ctx* ctx, const void* q_rot, const dapq_cache_view* cache,
                       const float* lse_in, float* scores, float* lse_out, float* syn_mass, void* stream) {
  if (!ctx) return DAPQ_ERR_INVALID_ARG;
  if (!q_rot || !scores) return fail(ctx, DAPQ_ERR_INVALID_ARG, "dapq_score: NULL argument");
  if (!aligned16(q_rot)) return fail(ctx, DAPQ_ERR_UNSUPPORTED, "q_rot must be 16-byte aligned");
  CacheDev cd;
  dapq_status st = check_view(ctx, cache, false, false, &cd);
  if (st != DAPQ_OK) return st;
  SeqTable t;
  st = build_table(ctx, cache->batch, cache->cu_rows_host, cache->prompt_len_host, nullptr, nullptr, nullptr, &t);
  if (st != DAPQ_OK) return st;
  DeviceGuard guard(ctx->device);
  if (wants_umma(ctx) && !syn_mass) {
    // the caller's bf16 queries are exact in bf16: one bf16 x bf16 MMA pass, no conversion of K
    if (wants_lo(ctx)) {
      UmmaPlan plan;
      if (umma_plan(q_rot, 0, 0, cd, t, ctx->dims, ctx->n_sm, &plan))
        return run_score_umma(ctx, plan, t, lse_in, scores, t.cu_prompt[t.batch], lse_out, (cudaStream_t)stream);
    } else {
      QgPlan plan;
      if (qg_plan(q_rot, 0, cd, t, ctx->dims, ctx->n_sm, &plan))
        return run_score_qg(ctx, plan, t, lse_in, scores, t.cu_prompt[t.batch], lse_out, false, (cudaStream_t)stream);
    }
  }
  return run_score(ctx, ctx->shape.dtype, q_rot, cd, t, lse_in, scores, t.cu_prompt[t.batch], lse_out, syn_mass, (cudaStream_t)stream);
}

dapq_status dapq_topk_select(dapq_ctx* ctx, const float* scores, const int32_t* cu_prompt_host,
                             const int32_t* k_keep_host, int32_t batch, int32_t* idx_out, void* stream) {
  if (!ctx) return DAPQ_ERR_INVALID_ARG;
  if (!scores || !cu_prompt_host || !k_keep_host || !idx_out)
    return fail(ctx, DAPQ_ERR_INVALID_ARG, "dapq_topk_select: NULL argument");
  SeqTable t;
  dapq_status st = build_table(ctx, batch, nullptr, nullptr, cu_prompt_host, k_keep_host, nullptr, &t);
  if (st != DAPQ_OK) return st;
  DeviceGuard guard(ctx->device);
  return run_select(ctx, scores, t.cu_prompt[batch], idx_out, t.cu_keep[batch], t, (cudaStream_t)stream);
}

dapq_status dapq_compact_kv(dapq_ctx* ctx, const dapq_cache_view* cache, const int32_t* idx,
                            const int32_t* k_keep_host, void* k_out, void* v_out, void* stream) {
  if (!ctx) return DAPQ_ERR_INVALID_ARG;
  if (!idx || !k_keep_host || !k_out || !v_out) return fail(ctx, DAPQ_ERR_INVALID_ARG, "dapq_compact_kv: NULL argument");
  if (!aligned16(k_out) || !aligned16(v_out)) return fail(ctx, DAPQ_ERR_UNSUPPORTED, "k_out / v_out must be 16-byte aligned");
  CacheDev cd;
  dapq_status st = check_view(ctx, cache, true, false, &cd);
  if (st != DAPQ_OK) return st;
  SeqTable t;
  st = build_table(ctx, cache->batch, cache->cu_rows_host, cache->prompt_len_host, nullptr, k_keep_host, nullptr, &t);
  if (st != DAPQ_OK) return st;
  DeviceGuard guard(ctx->device);
  cudaError_t e = launch_compact(ctx->shape.dtype, cd, idx, t.cu_keep[t.batch], k_out, v_out, t,
                                 ctx->dims.n_kv_heads, ctx->status, (cudaStream_t)stream, &ctx->log);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "compaction kernel");
  return DAPQ_OK;
}

dapq_status dapq_recall(dapq_ctx* ctx, const int32_t* idx_gold, const int32_t* idx_pred,
                        const int32_t* prompt_len_host, const int32_t* k_keep_host, int32_t batch,
                        float* recall_out, void* stream) {
  if (!ctx) return DAPQ_ERR_INVALID_ARG;
  if (!idx_gold || !idx_pred || !prompt_len_host || !k_keep_host || !recall_out)
    return fail(ctx, DAPQ_ERR_INVALID_ARG, "dapq_recall: NULL argument");
  SeqTable t;
  dapq_status st = build_table(ctx, batch, nullptr, prompt_len_host, nullptr, k_keep_host, nullptr, &t);
  if (st != DAPQ_OK) return st;
  DeviceGuard guard(ctx->device);
  cudaError_t e = launch_recall(idx_gold, idx_pred, t.cu_keep[batch], t, ctx->dims.n_kv_heads, recall_out,
                                (cudaStream_t)stream, &ctx->log);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "recall kernel");
  return DAPQ_OK;
}

namespace {

// after_own_compaction: the kernel before this call in `stream` is the compaction kernel of an
// earlier evict on the same context (the layers of dapq_evict_layers); the rotation then does
// not wait for it before it starts.
dapq_status evict_impl(dapq_ctx* ctx, const void* q_pre, const dapq_cache_view* cache, const int32_t* k_keep_host,
                       void* k_out, void* v_out, int32_t* idx_out, float* scores_out, void* stream,
                       bool after_own_compaction) {
  if (!ctx) return DAPQ_ERR_INVALID_ARG;
  if (!q_pre || !k_keep_host || !k_out || !v_out) return fail(ctx, DAPQ_ERR_INVALID_ARG, "dapq_evict: NULL argument");
  if (!aligned16(k_out) || !aligned16(v_out)) return fail(ctx, DAPQ_ERR_UNSUPPORTED, "k_out / v_out must be 16-byte aligned");
  CacheDev cd;
  dapq_status st = check_view(ctx, cache, true, false, &cd);
  if (st != DAPQ_OK) return st;
  SeqTable t;
  st = build_table(ctx, cache->batch, cache->cu_rows_host, cache->prompt_len_host, nullptr, k_keep_host, nullptr, &t);
  if (st != DAPQ_OK) return st;
  DeviceGuard guard(ctx->device);
  cudaStream_t s = (cudaStream_t)stream;
  float* scores = scores_out ? scores_out : ctx->scores;
  int32_t* idx = idx_out ? idx_out : ctx->idx;
  const int64_t score_stride = t.cu_prompt[t.batch], idx_stride = t.cu_keep[t.batch];
  UmmaPlan plan;
  QgPlan qplan;
  const int64_t lo_rows = ctx->q_rows_max;
  const int flags = ctx->shape.flags;
  cudaError_t e;
  if (wants_umma(ctx) && !wants_lo(ctx) && qg_plan(ctx->q_rot, (flags & DAPQ_FLAG_Q_BF16) ? 0 : 1, cd, t, ctx->dims, ctx->n_sm, &qplan)) {
    // tensor-core scorer: rotated queries rounded to fp16, K tiles converted to fp16 on their way to the MMAs
    // (DAPQ_FLAG_Q_BF16: queries rounded to bf16, no conversion)
    // (with fp16 queries the rotation also leaves, in lse2, every query's logit against the first key of its
    // sequence: the reference that sweep 1 measures the row's other logits against)
    const RopeRef ref = {(const __nv_bfloat16*)cd.k, cd.k_head_stride, cd.k_row_stride, ctx->lse2, ctx->dims.group};
    e = launch_rope(ctx->shape.dtype, qplan.q_is_f16 ? kRopeOutF16 : kRopeOutBf16, 0, q_pre, ctx->q_rot, ctx->inv_freq, t,
                    ctx->dims, after_own_compaction, s, &ctx->log, &ref);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "rope kernel");
    st = run_score_qg(ctx, qplan, t, nullptr, scores, score_stride, nullptr, true, s);
  } else if (wants_umma(ctx) && wants_lo(ctx) && umma_plan(ctx->q_rot, 1, lo_rows, cd, t, ctx->dims, ctx->n_sm, &plan)) {
    // older tensor-core scorer: rotated queries as a bf16 pair hi + lo, the lo part added by a second MMA
    // pass in the sweeps that the flags name
    plan.lo_sweep1 = (flags & DAPQ_FLAG_Q_LO_SWEEP1) ? 1 : 0;
    plan.lo_sweep2 = (flags & DAPQ_FLAG_Q_LO_SWEEP2) ? 1 : 0;
    e = launch_rope(ctx->shape.dtype, kRopeOutSplitBf16, lo_rows * kHeadDim, q_pre, ctx->q_rot, ctx->inv_freq, t,
                    ctx->dims, after_own_compaction, s, &ctx->log);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "rope kernel");
    st = run_score_umma(ctx, plan, t, nullptr, scores, score_stride, nullptr, s);
  } else {
    // CUDA-core scorer: reads the rotated queries unrounded (fp32)
    e = launch_rope(ctx->shape.dtype, kRopeOutF32, 0, q_pre, ctx->q_rot, ctx->inv_freq, t, ctx->dims, after_own_compaction, s,
                    &ctx->log);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "rope kernel");
    st = run_score(ctx, DAPQ_F32, ctx->q_rot, cd, t, nullptr, scores, score_stride, nullptr, nullptr, s);
  }
  if (st != DAPQ_OK) return st;
  st = run_select(ctx, scores, score_stride, idx, idx_stride, t, s);
  if (st != DAPQ_OK) return st;
  e = launch_compact(ctx->shape.dtype, cd, idx, idx_stride, k_out, v_out, t, ctx->dims.n_kv_heads, ctx->status, s, &ctx->log);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "compaction kernel");
  return DAPQ_OK;
}

}  // namespace

dapq_status dapq_evict(dapq_ctx* ctx, const void* q_pre, const dapq_cache_view* cache,
                       const int32_t* k_keep_host, void* k_out, void* v_out, int32_t* idx_out,
                       float* scores_out, void* stream) {
  return evict_impl(ctx, q_pre, cache, k_keep_host, k_out, v_out, idx_out, scores_out, stream, false);
}

dapq_status dapq_evict_layers(dapq_ctx* ctx, int32_t n_layers, const void* const* q_pre,
                              const dapq_cache_view* caches, const int32_t* k_keep_host,
                              int64_t k_keep_layer_stride, void* const* k_out, void* const* v_out,
                              int32_t* const* idx_out, void* stream) {
  if (!ctx) return DAPQ_ERR_INVALID_ARG;
  if (n_layers < 0 || k_keep_layer_stride < 0) return fail(ctx, DAPQ_ERR_INVALID_ARG, "dapq_evict_layers: negative count or stride");
  if (n_layers > 0 && (!q_pre || !caches || !k_keep_host || !k_out || !v_out))
    return fail(ctx, DAPQ_ERR_INVALID_ARG, "dapq_evict_layers: NULL argument");
  for (int32_t l = 0; l < n_layers; ++l) {
    const dapq_status st = evict_impl(ctx, q_pre[l], &caches[l], k_keep_host + (int64_t)l * k_keep_layer_stride, k_out[l],
                                      v_out[l], idx_out ? idx_out[l] : nullptr, nullptr, stream, l > 0);
    if (st != DAPQ_OK) return st;
  }
  return DAPQ_OK;
}

namespace {

// First use of a staging set: its buffers (V only when some caller's V cannot be read in place) and events.
dapq_status ensure_stage(dapq_ctx* ctx, int set, bool need_v) {
  const dapq_shape& sh = ctx->shape;
  dapq_ctx::HostStage& hs = ctx->hs[set];
  const size_t row_bytes = (size_t)kHeadDim * ctx->elem_bytes;
  const size_t cache_bytes = (size_t)sh.n_kv_heads * (size_t)sh.max_total_rows * row_bytes;
  if (!ctx->copy_stream) {
    DAPQ_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
    DAPQ_CUDA(ctx, cudaEventCreateWithFlags(&ctx->fork, cudaEventDisableTiming));
  }
  if (!hs.k) {
    DAPQ_CUDA(ctx, cudaMalloc(&hs.q, (size_t)sh.max_batch * sh.n_q_heads * sh.n_pseudo * row_bytes));
    DAPQ_CUDA(ctx, cudaMalloc(&hs.k, cache_bytes));
    DAPQ_CUDA(ctx, cudaMalloc(&hs.ko, cache_bytes));
    DAPQ_CUDA(ctx, cudaMalloc(&hs.vo, cache_bytes));
    DAPQ_CUDA(ctx, cudaMalloc(&hs.idx, (size_t)sh.n_kv_heads * (size_t)sh.max_total_rows * sizeof(int32_t)));
    DAPQ_CUDA(ctx, cudaEventCreateWithFlags(&hs.in_done, cudaEventDisableTiming));
    DAPQ_CUDA(ctx, cudaEventCreateWithFlags(&hs.out_done, cudaEventDisableTiming));
  }
  if (need_v && !hs.v) DAPQ_CUDA(ctx, cudaMalloc(&hs.v, cache_bytes));
  return DAPQ_OK;
}

// Device address of the caller's V if the compaction kernel can read it in place (page-locked, addressable
// by the device, 16-byte geometry), else NULL.
const void* mapped_v(dapq_ctx* ctx, const CacheDev& hv) {
  cudaPointerAttributes pa;
  const int per16 = 16 / ctx->elem_bytes;
  if (hv.v_row_stride % per16 || hv.v_head_stride % per16) return nullptr;
  if (cudaPointerGetAttributes(&pa, hv.v) == cudaSuccess && pa.type == cudaMemoryTypeHost && pa.devicePointer &&
      aligned16(pa.devicePointer))
    return pa.devicePointer;
  cudaGetLastError();
  return nullptr;
}

}  // namespace

namespace {
dapq_status evict_layers_host_impl(dapq_ctx* ctx, int32_t n_layers, const void* const* q_pre_host,
                                   const dapq_cache_view* caches_host, const int32_t* k_keep_host,
                                   int64_t k_keep_layer_stride, void* const* k_out_host, void* const* v_out_host,
                                   int32_t* const* idx_out_host, void* stream);
}  // namespace

dapq_status dapq_evict_layers_host(dapq_ctx* ctx, int32_t n_layers, const void* const* q_pre_host,
                                   const dapq_cache_view* caches_host, const int32_t* k_keep_host,
                                   int64_t k_keep_layer_stride, void* const* k_out_host, void* const* v_out_host,
                                   int32_t* const* idx_out_host, void* stream) {
  if (!ctx) return DAPQ_ERR_INVALID_ARG;
  const dapq_status st = evict_layers_host_impl(ctx, n_layers, q_pre_host, caches_host, k_keep_host, k_keep_layer_stride,
                                                k_out_host, v_out_host, idx_out_host, stream);
  if (st != DAPQ_OK) {
    // a layer failed with copies of earlier layers possibly still in flight: the caller's buffers may be
    // reused as soon as this call returns, so wait for both streams first (their own errors do not matter now)
    DeviceGuard guard(ctx->device);
    if (ctx->copy_stream) cudaStreamSynchronize(ctx->copy_stream);
    cudaStreamSynchronize((cudaStream_t)stream);
    cudaGetLastError();
  }
  return st;
}

namespace {
dapq_status evict_layers_host_impl(dapq_ctx* ctx, int32_t n_layers, const void* const* q_pre_host,
                                   const dapq_cache_view* caches_host, const int32_t* k_keep_host,
                                   int64_t k_keep_layer_stride, void* const* k_out_host, void* const* v_out_host,
                                   int32_t* const* idx_out_host, void* stream) {
  if (n_layers < 0 || k_keep_layer_stride < 0) return fail(ctx, DAPQ_ERR_INVALID_ARG, "dapq_evict_layers_host: negative count or stride");
  if (n_layers > 0 && (!q_pre_host || !caches_host || !k_keep_host || !k_out_host || !v_out_host))
    return fail(ctx, DAPQ_ERR_INVALID_ARG, "dapq_evict_layers_host: NULL argument");
  DeviceGuard guard(ctx->device);
  cudaStream_t s = (cudaStream_t)stream;
  const dapq_shape& sh = ctx->shape;
  const size_t eb = (size_t)ctx->elem_bytes, row_bytes = (size_t)kHeadDim * eb;
  bool forked = false;
  for (int32_t l = 0; l < n_layers; ++l) {
    const int32_t* keep = k_keep_host + (int64_t)l * k_keep_layer_stride;
    if (!q_pre_host[l] || !k_out_host[l] || !v_out_host[l]) return fail(ctx, DAPQ_ERR_INVALID_ARG, "dapq_evict_layers_host: NULL layer pointer");
    CacheDev hv;
    dapq_status st = check_view(ctx, &caches_host[l], true, true, &hv);
    if (st != DAPQ_OK) return st;
    SeqTable t;
    st = build_table(ctx, caches_host[l].batch, caches_host[l].cu_rows_host, caches_host[l].prompt_len_host, nullptr, keep,
                     nullptr, &t);
    if (st != DAPQ_OK) return st;
    const void* v_in_place = mapped_v(ctx, hv);
    const int set = l & 1;
    st = ensure_stage(ctx, set, v_in_place == nullptr);
    if (st != DAPQ_OK) return st;
    dapq_ctx::HostStage& hs = ctx->hs[set];
    cudaStream_t cs = ctx->copy_stream;
    if (!forked) {                                       // the copies start behind the work already in `stream`
      DAPQ_CUDA(ctx, cudaEventRecord(ctx->fork, s));
      DAPQ_CUDA(ctx, cudaStreamWaitEvent(cs, ctx->fork, 0));
      forked = true;
    }
    if (l >= 2) DAPQ_CUDA(ctx, cudaStreamWaitEvent(cs, hs.out_done, 0));   // the set's last user is done with it
    // ---- inputs: q and the used row range [cu_rows[0], cu_rows[B]) of every head of K, packed from row 0
    const int64_t row0 = t.cu_rows[0], n_rows = t.cu_rows[t.batch] - row0;
    DAPQ_CUDA(ctx, cudaMemcpyAsync(hs.q, q_pre_host[l], (size_t)t.batch * sh.n_q_heads * sh.n_pseudo * row_bytes,
                                   cudaMemcpyHostToDevice, cs));
    for (int h = 0; h < sh.n_kv_heads; ++h) {
      const char* ks = (const char*)hv.k + ((size_t)h * hv.k_head_stride + (size_t)row0 * hv.k_row_stride) * eb;
      DAPQ_CUDA(ctx, cudaMemcpy2DAsync((char*)hs.k + (size_t)h * n_rows * row_bytes, row_bytes, ks,
                                       (size_t)hv.k_row_stride * eb, row_bytes, (size_t)n_rows, cudaMemcpyHostToDevice, cs));
      if (v_in_place) continue;
      const char* vs = (const char*)hv.v + ((size_t)h * hv.v_head_stride + (size_t)row0 * hv.v_row_stride) * eb;
      DAPQ_CUDA(ctx, cudaMemcpy2DAsync((char*)hs.v + (size_t)h * n_rows * row_bytes, row_bytes, vs,
                                       (size_t)hv.v_row_stride * eb, row_bytes, (size_t)n_rows, cudaMemcpyHostToDevice, cs));
    }
    DAPQ_CUDA(ctx, cudaEventRecord(hs.in_done, cs));
    // ---- the layer itself, on the caller's stream
    int32_t cu_local[kMaxBatch + 1];
    for (int b = 0; b <= t.batch; ++b) cu_local[b] = (int32_t)(t.cu_rows[b] - row0);
    dapq_cache_view dv;
    memset(&dv, 0, sizeof(dv));
    dv.k = hs.k;
    dv.k_head_stride = n_rows * kHeadDim;
    dv.k_row_stride = kHeadDim;
    if (v_in_place) {
      dv.v = (const char*)v_in_place + (size_t)row0 * hv.v_row_stride * eb;   // row 0 of the view = row cu_rows[0] of the caller's
      dv.v_head_stride = hv.v_head_stride;
      dv.v_row_stride = hv.v_row_stride;
    } else {
      dv.v = hs.v;
      dv.v_head_stride = n_rows * kHeadDim;
      dv.v_row_stride = kHeadDim;
    }
    dv.cu_rows_host = cu_local;
    dv.prompt_len_host = caches_host[l].prompt_len_host;
    dv.batch = t.batch;
    DAPQ_CUDA(ctx, cudaStreamWaitEvent(s, hs.in_done, 0));
    st = dapq_evict(ctx, hs.q, &dv, keep, hs.ko, hs.vo, hs.idx, nullptr, stream);
    if (st != DAPQ_OK) return st;
    // ---- results
    const size_t kt = (size_t)t.cu_keep[t.batch];
    DAPQ_CUDA(ctx, cudaMemcpyAsync(k_out_host[l], hs.ko, (size_t)sh.n_kv_heads * kt * row_bytes, cudaMemcpyDeviceToHost, s));
    DAPQ_CUDA(ctx, cudaMemcpyAsync(v_out_host[l], hs.vo, (size_t)sh.n_kv_heads * kt * row_bytes, cudaMemcpyDeviceToHost, s));
    if (idx_out_host && idx_out_host[l])
      DAPQ_CUDA(ctx, cudaMemcpyAsync(idx_out_host[l], hs.idx, (size_t)sh.n_kv_heads * kt * sizeof(int32_t),
                                     cudaMemcpyDeviceToHost, s));
    DAPQ_CUDA(ctx, cudaEventRecord(hs.out_done, s));
  }
  DAPQ_CUDA(ctx, cudaStreamSynchronize(s));
  return DAPQ_OK;
}
}  // namespace

dapq_status dapq_evict_host(dapq_ctx* ctx, const void* q_pre_host, const dapq_cache_view* cache_host,
                            const int32_t* k_keep_host, void* k_out_host, void* v_out_host,
                            int32_t* idx_out_host, void* stream) {
  if (!ctx) return DAPQ_ERR_INVALID_ARG;
  if (!q_pre_host || !cache_host || !k_keep_host || !k_out_host || !v_out_host)
    return fail(ctx, DAPQ_ERR_INVALID_ARG, "dapq_evict_host: NULL argument");
  return dapq_evict_layers_host(ctx, 1, &q_pre_host, cache_host, k_keep_host, 0, &k_out_host, &v_out_host, &idx_out_host, stream);
}

}  // extern "C"
