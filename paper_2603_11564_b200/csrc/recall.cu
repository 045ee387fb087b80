// Recall of a predicted retained set against a gold one (Section 3.3, Eq. 1-3):
//   Recall_W = |M_gold ∩ M_pred| / |M_gold|
// per (sequence, KV head), where both sets are index lists as dapq_topk_select writes them
// (ascending, sequence-local).  One CTA per (sequence, KV head): every thread looks its gold
// indices up in the predicted list by binary search; the hits are counted with integer adds,
// so the result is exact.
#include "dapq_internal.cuh"

namespace dapq {
namespace {

constexpr int kRecallThreads = 256;

__global__ void __launch_bounds__(kRecallThreads)
recall_kernel(const int32_t* __restrict__ gold, const int32_t* __restrict__ pred, int64_t idx_stride,
              const __grid_constant__ SeqTable t, int n_kv_heads, float* __restrict__ recall) {
  __shared__ int warp_hits[kRecallThreads / 32];
  const int b = blockIdx.x, kvh = blockIdx.y;
  const int k0 = t.cu_keep[b], K = t.cu_keep[b + 1] - k0;
  const int32_t* g = gold + (int64_t)kvh * idx_stride + k0;
  const int32_t* p = pred + (int64_t)kvh * idx_stride + k0;
  int hits = 0;
  for (int r = threadIdx.x; r < K; r += kRecallThreads) {
    const int32_t want = g[r];
    int lo = 0, hi = K;                                   // first position with p[pos] >= want
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (p[mid] < want) lo = mid + 1; else hi = mid;
    }
    hits += (lo < K && p[lo] == want) ? 1 : 0;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) hits += __shfl_xor_sync(0xffffffffu, hits, o);
  if ((threadIdx.x & 31) == 0) warp_hits[threadIdx.x >> 5] = hits;
  __syncthreads();
  if (threadIdx.x == 0) {
    int total = 0;
    for (int w = 0; w < kRecallThreads / 32; ++w) total += warp_hits[w];
    recall[(int64_t)b * n_kv_heads + kvh] = (float)total / (float)K;
  }
}

}  // namespace

cudaError_t launch_recall(const int32_t* gold, const int32_t* pred, int64_t idx_stride, const SeqTable& t,
                          int n_kv_heads, float* recall, cudaStream_t s, LaunchLog* log) {
  log->begin(kKindRecall, s);
  recall_kernel<<<dim3(t.batch, n_kv_heads), kRecallThreads, 0, s>>>(gold, pred, idx_stride, t, n_kv_heads, recall);
  log->end(s);
  return cudaGetLastError();
}

}  // namespace dapq
