// Optional pooling of the accumulated scores before selection.  The paper specifies none for
// DapQ; it describes the SnapKV / PyramidKV baselines as selecting on pooled accumulated
// attention scores (Sections 2 and 5.1), and this kernel offers the same step: a 1-D window of
// odd width centred on each prompt position, stride 1, clipped at the ends of the sequence;
// the maximum, or the mean of the positions that exist.
//
// One CTA per 1024 positions of a (sequence, KV head); the tile and its halo are staged in
// shared memory.  The mean is summed left to right, so the result is deterministic.  The
// scores of a layer are a few MB and L2-resident: the kernel is latency-bound.
#include <math_constants.h>

#include "dapq_internal.cuh"

namespace dapq {
namespace {

constexpr int kPoolThreads = 256;
constexpr int kPoolTile = 1024;
constexpr int kMaxHalo = DAPQ_MAX_POOL_KERNEL / 2;

__global__ void __launch_bounds__(kPoolThreads)
pool_scores_kernel(const float* __restrict__ scores, float* __restrict__ pooled, int64_t stride,
                   const __grid_constant__ SeqTable t, const __grid_constant__ ChunkTable tiles, int kernel, int mode) {
  __shared__ float tile[kPoolTile + 2 * kMaxHalo];
  pdl_wait();
  const int b = find_segment(tiles.cu_chunk, t.batch, blockIdx.x);
  const int L = t.prompt_len[b], r = kernel / 2;
  const int j0 = (blockIdx.x - tiles.cu_chunk[b]) * kPoolTile;          // first position of this tile
  const float* x = scores + (int64_t)blockIdx.y * stride + t.cu_prompt[b];
  float* y = pooled + (int64_t)blockIdx.y * stride + t.cu_prompt[b];
  const int lo = max(0, j0 - r), hi = min(L, j0 + kPoolTile + r);       // staged range [lo, hi)
  for (int j = lo + threadIdx.x; j < hi; j += kPoolThreads) tile[j - lo] = x[j];
  __syncthreads();
  for (int j = j0 + threadIdx.x; j < min(L, j0 + kPoolTile); j += kPoolThreads) {
    const int w0 = max(0, j - r), w1 = min(L, j + r + 1);
    float acc = mode == DAPQ_POOL_MAX ? -CUDART_INF_F : 0.f;
    for (int k = w0; k < w1; ++k) {
      const float v = tile[k - lo];
      acc = mode == DAPQ_POOL_MAX ? fmaxf(acc, v) : acc + v;
    }
    y[j] = mode == DAPQ_POOL_MAX ? acc : acc / (float)(w1 - w0);
  }
}

}  // namespace

cudaError_t launch_pool(const float* scores, float* pooled, int64_t stride, const SeqTable& t, int n_kv_heads,
                        int kernel, int mode, cudaStream_t s, LaunchLog* log) {
  ChunkTable tiles;
  tiles.chunk_tiles = 1;
  int32_t n = 0;
  for (int b = 0; b < t.batch; ++b) {
    tiles.cu_chunk[b] = n;
    n += (t.prompt_len[b] + kPoolTile - 1) / kPoolTile;
  }
  tiles.cu_chunk[t.batch] = n;
  tiles.n_chunks = n;
  log->begin(kKindPool, s);
  launch_pdl(pool_scores_kernel, dim3(n, n_kv_heads), dim3(kPoolThreads), 0, s, 1, scores, pooled, stride, t, tiles, kernel, mode);
  log->end(s);
  return cudaGetLastError();
}

}  // namespace dapq
