// dapq_score_static: the CUDA-core scorer for callers that must not allocate.
//
// Some callers of this library cannot call cudaMalloc at the point where they need scores:
// code that runs inside a memory-pool-managed region of a serving engine whose allocator owns
// every byte of the device, plug-ins loaded into a process that forbids driver allocations
// after start-up, or anything that runs between a pool snapshot and its restore.  dapq_create
// allocates a workspace, so those callers cannot even make a context.  This entry point needs
// none: the scorer's scratch (the per-chunk running max / sum partials of the first sweep and
// the merged log-sum-exp) lives in a fixed array that is part of the library image on every
// device that loads it.  The price is a hard size limit and one shared scratch area.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <mutex>

#include "dapq_internal.cuh"

using namespace dapq;

namespace {

// The scratch itself.  In host code this name is only a handle for the runtime (it is not a
// device address); the address each device uses is looked up once with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[DAPQ_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices] = {};     // per device, filled on the first call on that device

dapq_status fail_static(char* err, size_t err_len, dapq_status st, const char* fmt, ...) {
  if (err && err_len) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(err, err_len, fmt, ap);
    va_end(ap);
  }
  return st;
}

struct DeviceScope {
  int prev = -1;
  bool ok = true;
  explicit DeviceScope(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceScope() { if (prev >= 0) cudaSetDevice(prev); }
};

}  // namespace

extern "C" dapq_status dapq_score_static(const dapq_shape* sh, int device, const void* q_rot,
                                          const dapq_cache_view* cv, float* scores, void* stream,
                                          char* err, size_t err_len) {
  if (err && err_len) err[0] = '\0';
  if (!sh || !q_rot || !cv || !scores) return fail_static(err, err_len, DAPQ_ERR_INVALID_ARG, "dapq_score_static: NULL argument");
  if (sh->head_dim != kHeadDim) return fail_static(err, err_len, DAPQ_ERR_UNSUPPORTED, "head_dim must be 128");
  if (sh->n_pseudo < 1 || sh->n_pseudo > kMaxPseudo) return fail_static(err, err_len, DAPQ_ERR_UNSUPPORTED, "n_pseudo must be in 1..128");
  if (sh->n_q_heads < 1 || sh->n_kv_heads < 1 || sh->n_q_heads % sh->n_kv_heads)
    return fail_static(err, err_len, DAPQ_ERR_INVALID_ARG, "n_kv_heads must divide n_q_heads");
  if (sh->dtype != DAPQ_BF16 && sh->dtype != DAPQ_F32) return fail_static(err, err_len, DAPQ_ERR_INVALID_ARG, "unknown dtype");
  if (!(sh->softmax_scale >= 0.f)) return fail_static(err, err_len, DAPQ_ERR_INVALID_ARG, "softmax_scale must be >= 0");
  if (device < 0 || device >= kMaxDevices) return fail_static(err, err_len, DAPQ_ERR_INVALID_ARG, "device %d out of range", device);
  if (!cv->k || !cv->cu_rows_host || !cv->prompt_len_host || cv->reserved != 0)
    return fail_static(err, err_len, DAPQ_ERR_INVALID_ARG, "cache view needs k, cu_rows_host, prompt_len_host; reserved must be 0");
  if (cv->batch < 1 || cv->batch > kMaxBatch) return fail_static(err, err_len, DAPQ_ERR_INVALID_ARG, "batch must be in 1..128");
  const int elem_bytes = sh->dtype == DAPQ_BF16 ? 2 : 4, per16 = 16 / elem_bytes;
  if (cv->k_row_stride < kHeadDim || cv->k_head_stride < 0)
    return fail_static(err, err_len, DAPQ_ERR_INVALID_ARG, "row stride must be >= head_dim and head stride >= 0");
  if (cv->k_row_stride % per16 || cv->k_head_stride % per16 || (reinterpret_cast<uintptr_t>(cv->k) & 15u) ||
      (reinterpret_cast<uintptr_t>(q_rot) & 15u))
    return fail_static(err, err_len, DAPQ_ERR_UNSUPPORTED, "q_rot, K and the K strides must be multiples of 16 bytes");

  // ---- sequence table and the scratch this call needs
  SeqTable t;
  memset(&t, 0, sizeof(t));
  t.batch = cv->batch;
  int64_t rows = cv->cu_rows_host[0], prompt = 0, chunks = 0;
  if (rows < 0) return fail_static(err, err_len, DAPQ_ERR_INVALID_ARG, "cu_rows[0] is negative");
  for (int b = 0; b < cv->batch; ++b) {
    const int64_t L = cv->prompt_len_host[b];
    if (L < 1) return fail_static(err, err_len, DAPQ_ERR_INVALID_ARG, "prompt length of sequence %d must be >= 1", b);
    if ((int64_t)cv->cu_rows_host[b + 1] - cv->cu_rows_host[b] != L + sh->n_pseudo)
      return fail_static(err, err_len, DAPQ_ERR_INVALID_ARG, "sequence %d does not own L_b + N cache rows", b);
    t.cu_rows[b] = cv->cu_rows_host[b];
    t.cu_rows[b + 1] = cv->cu_rows_host[b + 1];
    t.prompt_len[b] = (int32_t)L;
    t.pos_start[b] = (int32_t)L;
    t.cu_prompt[b] = (int32_t)prompt;
    t.cu_keep[b] = (int32_t)prompt;
    prompt += L;
    chunks += (L + kChunkKeys - 1) / kChunkKeys + 1;
    if (prompt > 0x7fffffffLL) return fail_static(err, err_len, DAPQ_ERR_UNSUPPORTED, "more than 2^31 prompt rows");
  }
  t.cu_prompt[cv->batch] = (int32_t)prompt;
  t.cu_keep[cv->batch] = (int32_t)prompt;
  // layout of the fixed area: the base-2 lse [B, H_q, N] first, the sweeps' partials after it
  const size_t hq_n = (size_t)sh->n_q_heads * sh->n_pseudo;
  const size_t part_off = ((size_t)cv->batch * hq_n * sizeof(float) + 255) & ~(size_t)255;
  const size_t need = part_off + (size_t)chunks * hq_n * sizeof(float2);
  if (need > (size_t)DAPQ_STATIC_SCRATCH_BYTES)
    return fail_static(err, err_len, DAPQ_ERR_WORKSPACE,
                       "dapq_score_static: this call needs %zu bytes of scratch, the fixed area holds %d "
                       "(round_up(B x H_q x N x 4, 256) + sum_b (ceil(L_b / 512) + 1) x H_q x N x 8 bytes); use "
                       "dapq_create + dapq_score for larger caches",
                       need, (int)DAPQ_STATIC_SCRATCH_BYTES);
  // what is left lets the launcher cut small inputs into finer chunks
  const int64_t max_chunks = (int64_t)(((size_t)DAPQ_STATIC_SCRATCH_BYTES - part_off) / (hq_n * sizeof(float2)));

  DeviceScope scope(device);
  if (!scope.ok) return fail_static(err, err_len, DAPQ_ERR_CUDA, "cannot make device %d current", device);
  void* base = nullptr;
  {
    // set-up, once per device, with that device current: resolve the array's device address (this loads the
    // module that holds the array)
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[device]) {
      void* p = nullptr;
      const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
      if (e != cudaSuccess || !p)
        return fail_static(err, err_len, DAPQ_ERR_CUDA, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
      // ... and bring the code of every kernel this entry point can launch to the device now, so that no later
      // call has to (a kernel's first use loads its code, which takes device memory)
      const cudaError_t e2 = score_fma_preload();
      if (e2 != cudaSuccess)
        return fail_static(err, err_len, DAPQ_ERR_CUDA, "loading the score kernels: %s", cudaGetErrorString(e2));
      g_scratch_addr[device] = p;
    }
    base = g_scratch_addr[device];
  }

  Dims dm;
  dm.n_q_heads = sh->n_q_heads;
  dm.n_kv_heads = sh->n_kv_heads;
  dm.group = sh->n_q_heads / sh->n_kv_heads;
  dm.n_pseudo = sh->n_pseudo;
  const double scale = sh->softmax_scale > 0.f ? (double)sh->softmax_scale : 1.0 / sqrt((double)kHeadDim);
  dm.scale_log2e = (float)(scale * 1.4426950408889634074);
  CacheDev cd;
  cd.k = cv->k;
  cd.v = nullptr;
  cd.k_head_stride = cv->k_head_stride;
  cd.k_row_stride = cv->k_row_stride;
  cd.v_head_stride = cd.v_row_stride = 0;
  // Every partial and every lse entry the second sweep reads is written by this call first,
  // so nothing left in the area by an earlier call has to be cleared.
  float* lse2 = reinterpret_cast<float*>(base);
  float2* part = reinterpret_cast<float2*>(static_cast<unsigned char*>(base) + part_off);
  int n_sm = 0;
  if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || n_sm < 1)
    return fail_static(err, err_len, DAPQ_ERR_CUDA, "cannot query device %d", device);
  LaunchLog log;
  const cudaError_t e = launch_score_fma(sh->dtype, sh->dtype, q_rot, cd, t, dm, nullptr, part, max_chunks, n_sm, lse2, scores,
                                         (int64_t)prompt, nullptr, nullptr, (cudaStream_t)stream, &log);
  if (e != cudaSuccess) return fail_static(err, err_len, DAPQ_ERR_CUDA, "score kernels: %s", cudaGetErrorString(e));
  return DAPQ_OK;
}
