// Per-head selection of the retained tokens (Section 4.2, Eq. 5: M_retain = TopK_j S(j)).
//
// One CTA per (sequence, KV head).  A 4-pass, 8-bit radix select over the order-preserving
// integer image of the fp32 scores finds the exact bit pattern of the K-th largest score
// and how many entries equal to it still fit; an ordered compaction then writes, in
// ascending position, every entry above the threshold plus the lowest-position ties.
// Integer work only: the result is exact and deterministic.
#include "dapq_internal.cuh"

namespace dapq {
namespace {

constexpr int kTopkThreads = 1024;
constexpr int kWarps = kTopkThreads / 32;

// Monotone map float -> uint32 (larger float <=> larger key), valid for all finite values.
__device__ __forceinline__ uint32_t order_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__global__ void __launch_bounds__(kTopkThreads)
topk_select_kernel(const float* __restrict__ scores, int64_t score_stride, int32_t* __restrict__ idx,
                   int64_t idx_stride, const __grid_constant__ SeqTable t) {
  __shared__ uint32_t hist[256];
  __shared__ uint32_t s_prefix, s_remaining;
  __shared__ uint32_t cnt_gt[kWarps], cnt_eq[kWarps];

  const int b = blockIdx.x, kvh = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int L = t.prompt_len[b];
  const int K = t.cu_keep[b + 1] - t.cu_keep[b];
  const float* x = scores + (int64_t)kvh * score_stride + t.cu_prompt[b];
  int32_t* out = idx + (int64_t)kvh * idx_stride + t.cu_keep[b];

  if (K >= L) {                      // keep everything
    for (int j = tid; j < L; j += kTopkThreads) out[j] = j;
    return;
  }

  if (tid == 0) { s_prefix = 0u; s_remaining = (uint32_t)K; }
  const int L_pad = (L + kTopkThreads - 1) / kTopkThreads * kTopkThreads;

  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    const uint32_t hi_mask = (pass == 0) ? 0u : (0xffffffffu << (shift + 8));
    for (int d = tid; d < 256; d += kTopkThreads) hist[d] = 0u;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    for (int j = tid; j < L_pad; j += kTopkThreads) {
      uint32_t digit = 0xffffffffu;                       // sentinel: not a candidate
      if (j < L) {
        const uint32_t key = order_key(x[j]);
        if ((key & hi_mask) == prefix) digit = (key >> shift) & 255u;
      }
      // one shared-memory atomic per distinct digit in the warp (scores of one head share
      // their exponent, so most lanes hit the same bin)
      const uint32_t peers = __match_any_sync(0xffffffffu, digit);
      if (digit != 0xffffffffu && lane == __ffs(peers) - 1) atomicAdd(&hist[digit], __popc(peers));
    }
    __syncthreads();
    if (warp == 0) {
      // lane l owns bins 255-8l .. 248-8l (descending); find the bin holding the K-th largest
      const uint32_t remaining = s_remaining;
      uint32_t local[8], sum = 0u;
#pragma unroll
      for (int e = 0; e < 8; ++e) { local[e] = hist[255 - 8 * lane - e]; sum += local[e]; }
      uint32_t incl = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
      }
      const uint32_t hit = __ballot_sync(0xffffffffu, incl >= remaining);
      const int owner = __ffs(hit) - 1;                   // exists: candidates >= remaining
      if (lane == owner) {
        uint32_t cum = incl - sum;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          if (cum + local[e] >= remaining) {
            s_prefix = prefix | ((uint32_t)(255 - 8 * lane - e) << shift);
            s_remaining = remaining - cum;
            break;
          }
          cum += local[e];
        }
      }
    }
    __syncthreads();
  }

  const uint32_t thr = s_prefix;          // key of the K-th largest score
  const uint32_t n_ties = s_remaining;    // entries equal to it that are kept (lowest positions)

  // ordered compaction: warp w owns the contiguous span [w * span, (w+1) * span)
  const int span = ((L + kWarps - 1) / kWarps + 31) / 32 * 32;
  const int j0 = warp * span, j1 = min(L, j0 + span);
  uint32_t n_gt = 0u, n_eq = 0u;
  for (int j = j0 + lane; j < j0 + span; j += 32) {
    const uint32_t key = (j < j1) ? order_key(x[j]) : 0u;
    n_gt += __popc(__ballot_sync(0xffffffffu, j < j1 && key > thr));
    n_eq += __popc(__ballot_sync(0xffffffffu, j < j1 && key == thr));
  }
  if (lane == 0) { cnt_gt[warp] = n_gt; cnt_eq[warp] = n_eq; }
  __syncthreads();
  uint32_t gt_before = 0u, eq_before = 0u;
  for (int w = 0; w < warp; ++w) { gt_before += cnt_gt[w]; eq_before += cnt_eq[w]; }
  uint32_t pos = gt_before + min(eq_before, n_ties);
  const uint32_t lt_mask = (1u << lane) - 1u;
  for (int j = j0 + lane; j < j0 + span; j += 32) {
    const uint32_t key = (j < j1) ? order_key(x[j]) : 0u;
    const bool gt = j < j1 && key > thr;
    const bool eq = j < j1 && key == thr;
    const uint32_t eq_bal = __ballot_sync(0xffffffffu, eq);
    const bool take = gt || (eq && eq_before + __popc(eq_bal & lt_mask) < n_ties);
    const uint32_t take_bal = __ballot_sync(0xffffffffu, take);
    if (take) out[pos + __popc(take_bal & lt_mask)] = j;
    pos += __popc(take_bal);
    eq_before += __popc(eq_bal);
  }
}

}  // namespace

cudaError_t launch_topk(const float* scores, int64_t score_stride, int32_t* idx, int64_t idx_stride,
                        const SeqTable& t, int n_kv_heads, cudaStream_t s, LaunchLog* log) {
  log->begin(kKindTopk, s);
  topk_select_kernel<<<dim3(t.batch, n_kv_heads), kTopkThreads, 0, s>>>(scores, score_stride, idx,
                                                                        idx_stride, t);
  log->end(s);
  return cudaGetLastError();
}

}  // namespace dapq
