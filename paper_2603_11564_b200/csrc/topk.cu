// Per-head selection of the retained tokens (Section 4.2, Eq. 5: M_retain = TopK_j S(j)).
//
// One thread-block cluster of 1, 2, 4 or 8 CTAs (by the longest sequence: 4k to 16k keys per
// CTA, fewer CTAs when the grid would not fit one wave) per (sequence, KV head).  Each CTA owns a contiguous
// slice of the head's scores and keeps their order-preserving integer images in shared
// memory, so the scores are read from global memory once.  A 3-pass radix select (11 + 11 +
// 10 bits, most significant first) finds the exact bit pattern of the K-th largest score and
// how many entries equal to it still fit: per pass every CTA histograms its slice with plain
// shared-memory atomics, adds its non-empty bins into the table of EVERY CTA of the cluster
// through distributed shared memory (remote adds need no reply), and after one cluster barrier
// scans its own copy of the merged table for the digit that holds the K-th entry.  After the
// first pass a CTA keeps only its candidates (the keys of the selected bin) in a short list, so
// the later passes touch few keys.  An ordered compaction then writes, in ascending position,
// every entry above the threshold plus the lowest-position ties; the CTAs push their counts to
// each other the same way, so no CTA reads remote memory and none has to outlive another.
// Integer work only: the result is exact and deterministic.
#include <cooperative_groups.h>

#include "dapq_internal.cuh"

namespace cg = cooperative_groups;

namespace dapq {
namespace {

constexpr int kTopkThreads = 1024;
constexpr int kWarps = kTopkThreads / 32;
constexpr int kCluster = 8;                   // most CTAs per (sequence, head); portable cluster size
constexpr int kKeysPerCta = 4096;             // a CTA owns about this many keys, twice or four times as many
constexpr int kWaveCtas = 296;                // when the grid would otherwise exceed one wave (2 CTAs per SM)
constexpr int kBins = 2048;                   // 11-bit digits (the last pass uses 1024 of them)
constexpr int kMaxSliceSmem = 36864;          // keys a CTA can cache (144 KB); longer slices re-read global
constexpr int kMaxCand = 4096;                // candidate keys a CTA lists after the first pass

// Monotone map float -> uint32 (larger float <=> larger key), valid for all finite values.
__device__ __forceinline__ uint32_t order_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct TopkSmem {
  uint32_t merged[3][kBins];   // cluster-wide histogram of each pass (every CTA holds a copy)
  uint32_t hist[kBins];        // this CTA's histogram (all zero between passes)
  uint32_t cand[kMaxCand];     // this CTA's keys that share the first pass's digit
  uint32_t warp_sum[kWarps];
  uint32_t cnt_gt[kWarps], cnt_eq[kWarps];
  uint32_t peer_gt[kCluster], peer_eq[kCluster];   // totals of every CTA of the cluster, pushed by their owners
  uint32_t prefix, remaining, n_cand, list_ok;
};

// Adds this CTA's non-empty bins into the merged table of every CTA of the cluster and leaves the local table
// clear; local_bins keeps the thread's own two counts (the first pass's decide whether the candidates fit the list).
__device__ __forceinline__ void push_bins(TopkSmem& sm, uint32_t* const (&peer_merged)[kCluster], int n_cta, int pass,
                                          int tid, uint32_t (&local_bins)[kBins / kTopkThreads]) {
#pragma unroll
  for (int e = 0; e < kBins / kTopkThreads; ++e) {
    const int d = tid + e * kTopkThreads;
    const uint32_t c = sm.hist[d];
    local_bins[e] = c;
    if (c) {
      sm.hist[d] = 0u;
#pragma unroll
      for (int p = 0; p < kCluster; ++p)
        if (p < n_cta) atomicAdd(peer_merged[p] + pass * kBins + d, c);
    }
  }
}

// Scans the merged table of `pass` from the top digit down for the digit that holds the K-th entry (thread t owns
// digits 2047-2t and 2046-2t); extends sm.prefix by it and reduces sm.remaining to the rank within that digit.
__device__ __forceinline__ void select_digit(TopkSmem& sm, int pass, int shift, uint32_t prefix, int tid, int lane, int warp) {
  const uint32_t remaining = sm.remaining;
  const int d_hi = kBins - 1 - 2 * tid;
  const uint32_t v0 = sm.merged[pass][d_hi], v1 = sm.merged[pass][d_hi - 1];
  const uint32_t mine = v0 + v1;
  uint32_t incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) sm.warp_sum[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const uint32_t ws = sm.warp_sum[lane];
    uint32_t wi = ws;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += y;
    }
    sm.warp_sum[lane] = wi - ws;                         // exclusive prefix of the warp sums
  }
  __syncthreads();
  incl += sm.warp_sum[warp];
  const uint32_t excl = incl - mine;
  if (excl < remaining && incl >= remaining) {           // exactly one thread
    const bool first = excl + v0 >= remaining;
    sm.prefix = prefix | ((uint32_t)(first ? d_hi : d_hi - 1) << shift);
    sm.remaining = remaining - excl - (first ? 0u : v0);
  }
  __syncthreads();
}

__global__ void __launch_bounds__(kTopkThreads)
topk_select_kernel(const float* __restrict__ scores, int64_t score_stride, int32_t* __restrict__ idx,
                   int64_t idx_stride, const __grid_constant__ SeqTable t, int cache_keys) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  TopkSmem& sm = *reinterpret_cast<TopkSmem*>(smem_raw);
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw + sizeof(TopkSmem));   // [cache_keys]

  pdl_trigger();
  pdl_wait();
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int n_cta = (int)cluster.num_blocks();               // CTAs of this cluster (1, 2, 4 or 8)
  const int b = blockIdx.x / n_cta, kvh = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int L = t.prompt_len[b];
  const int K = t.cu_keep[b + 1] - t.cu_keep[b];
  const float* x = scores + (int64_t)kvh * score_stride + t.cu_prompt[b];
  int32_t* out = idx + (int64_t)kvh * idx_stride + t.cu_keep[b];

  // slice of this CTA: [j0, j1), a multiple of 32 keys long so that warps stay converged
  const int slice = (((L + n_cta - 1) / n_cta) + 31) & ~31;
  const int j0 = min(L, rank * slice), j1 = min(L, j0 + slice);
  const int n_own = j1 - j0;

  if (K >= L) {                      // keep everything (uniform over the cluster: no barrier is skipped by a part of it)
    for (int j = j0 + tid; j < j1; j += kTopkThreads) out[j] = j;
    return;
  }

  const bool cached = slice <= cache_keys;
  for (int d = tid; d < 3 * kBins; d += kTopkThreads) (&sm.merged[0][0])[d] = 0u;
  for (int d = tid; d < kBins; d += kTopkThreads) sm.hist[d] = 0u;
  if (tid == 0) { sm.prefix = 0u; sm.remaining = (uint32_t)K; sm.n_cand = 0u; }
  if (cached) {
    for (int j = tid; j < n_own; j += kTopkThreads) keys[j] = order_key(x[j0 + j]);
  }
  cluster.sync();                    // every CTA of the cluster runs and has cleared its tables

  uint32_t* peer_merged[kCluster];
#pragma unroll
  for (int p = 0; p < kCluster; ++p) peer_merged[p] = cluster.map_shared_rank(&sm.merged[0][0], p < n_cta ? p : 0);
  bool listed = false;               // the later passes read the candidate list instead of the slice

  for (int pass = 0; pass < 3; ++pass) {
    const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
    const uint32_t digit_mask = pass == 2 ? 1023u : 2047u;
    const uint32_t hi_mask = pass == 0 ? 0u : (pass == 1 ? 0xffe00000u : 0xfffffc00u);
    const uint32_t prefix = sm.prefix;
    const int n_scan = listed ? (int)sm.n_cand : n_own;
    for (int j = tid; j < n_scan; j += kTopkThreads) {
      const uint32_t key = listed ? sm.cand[j] : (cached ? keys[j] : order_key(x[j0 + j]));
      if ((key & hi_mask) == prefix) atomicAdd(&sm.hist[(key >> shift) & digit_mask], 1u);
    }
    __syncthreads();
    uint32_t local_bins[kBins / kTopkThreads];
    push_bins(sm, peer_merged, n_cta, pass, tid, local_bins);
    cluster.sync();
    select_digit(sm, pass, shift, prefix, tid, lane, warp);
    if (pass == 0) {
      // keep only this CTA's keys of the selected bin, if they fit the list (their number is
      // this CTA's own count of that bin, which the owner of the bin still holds)
      const uint32_t digit0 = sm.prefix >> 21;
#pragma unroll
      for (int e = 0; e < kBins / kTopkThreads; ++e)
        if ((uint32_t)(tid + e * kTopkThreads) == digit0) sm.list_ok = local_bins[e] <= (uint32_t)kMaxCand;
      __syncthreads();
      listed = sm.list_ok != 0u;           // (a flag of its own: n_cand starts to move as soon as the first thread lists)
      if (listed) {
        for (int j = tid; j < n_own; j += kTopkThreads) {
          const uint32_t key = cached ? keys[j] : order_key(x[j0 + j]);
          if ((key >> 21) == digit0) sm.cand[atomicAdd(&sm.n_cand, 1u)] = key;
        }
      }
      __syncthreads();
    }
  }

  const uint32_t thr = sm.prefix;          // key of the K-th largest score
  const uint32_t n_ties = sm.remaining;    // entries equal to it that are kept (lowest positions)

  // ordered compaction: within the CTA, warp w owns the contiguous span [w * span, (w+1) * span)
  const int span = (((n_own + kWarps - 1) / kWarps) + 31) & ~31;
  const int s0 = min(n_own, warp * span), s1 = min(n_own, s0 + span);
  uint32_t n_gt = 0u, n_eq = 0u;
  for (int j = s0 + lane; j < s0 + span; j += 32) {
    const uint32_t key = (j < s1) ? (cached ? keys[j] : order_key(x[j0 + j])) : 0u;
    n_gt += __popc(__ballot_sync(0xffffffffu, j < s1 && key > thr));
    n_eq += __popc(__ballot_sync(0xffffffffu, j < s1 && key == thr));
  }
  if (lane == 0) { sm.cnt_gt[warp] = n_gt; sm.cnt_eq[warp] = n_eq; }
  __syncthreads();
  if (warp == 0) {
    uint32_t g = sm.cnt_gt[lane], e = sm.cnt_eq[lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      g += __shfl_xor_sync(0xffffffffu, g, o);
      e += __shfl_xor_sync(0xffffffffu, e, o);
    }
    if (lane < n_cta) {                                    // lane p tells CTA p this CTA's totals
      *cluster.map_shared_rank(&sm.peer_gt[rank], lane) = g;
      *cluster.map_shared_rank(&sm.peer_eq[rank], lane) = e;
    }
  }
  cluster.sync();                    // the last remote access of the kernel is behind every CTA
  uint32_t gt_before = 0u, eq_before = 0u;
  for (int r = 0; r < rank; ++r) { gt_before += sm.peer_gt[r]; eq_before += sm.peer_eq[r]; }
  for (int w = 0; w < warp; ++w) { gt_before += sm.cnt_gt[w]; eq_before += sm.cnt_eq[w]; }
  uint32_t pos = gt_before + min(eq_before, n_ties);
  const uint32_t lt_mask = (1u << lane) - 1u;
  for (int j = s0 + lane; j < s0 + span; j += 32) {
    const uint32_t key = (j < s1) ? (cached ? keys[j] : order_key(x[j0 + j])) : 0u;
    const bool gt = j < s1 && key > thr;
    const bool eq = j < s1 && key == thr;
    const uint32_t eq_bal = __ballot_sync(0xffffffffu, eq);
    const bool take = gt || (eq && eq_before + __popc(eq_bal & lt_mask) < n_ties);
    const uint32_t take_bal = __ballot_sync(0xffffffffu, take);
    if (take) out[pos + __popc(take_bal & lt_mask)] = j0 + j;
    pos += __popc(take_bal);
    eq_before += __popc(eq_bal);
  }
}

// The same selection for slices of up to 16k keys per CTA (sequences of up to 128k keys): thread t of CTA r owns the
// kKpt CONSECUTIVE keys from position (r * 1024 + t) * kKpt and holds them in registers, so every scan is an
// unrolled register loop, and the final order (ascending position) is the thread order: one block-wide prefix
// sum of the threads' counts places every kept entry, no per-key ballots.  The first cluster barrier is split:
// a CTA arrives once its tables are clear and waits only before its first remote add.
template <int kKpt>
__global__ void __launch_bounds__(kTopkThreads)
topk_select_reg_kernel(const float* __restrict__ scores, int64_t score_stride, int32_t* __restrict__ idx,
                       int64_t idx_stride, const __grid_constant__ SeqTable t) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  TopkSmem& sm = *reinterpret_cast<TopkSmem*>(smem_raw);

  pdl_trigger();
  pdl_wait();
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int n_cta = (int)cluster.num_blocks();
  const int b = blockIdx.x / n_cta, kvh = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int L = t.prompt_len[b];
  const int K = t.cu_keep[b + 1] - t.cu_keep[b];
  const float* x = scores + (int64_t)kvh * score_stride + t.cu_prompt[b];
  int32_t* out = idx + (int64_t)kvh * idx_stride + t.cu_keep[b];

  const int base = (rank * kTopkThreads + tid) * kKpt;          // position of this thread's first key
  const int nv = max(0, min(kKpt, L - base));                   // how many of its keys exist
  if (K >= L) {                      // keep everything (uniform over the cluster)
    for (int e = 0; e < nv; ++e) out[base + e] = base + e;
    return;
  }

  for (int d = tid; d < 3 * kBins; d += kTopkThreads) (&sm.merged[0][0])[d] = 0u;
  for (int d = tid; d < kBins; d += kTopkThreads) sm.hist[d] = 0u;
  if (tid == 0) { sm.prefix = 0u; sm.remaining = (uint32_t)K; sm.n_cand = 0u; }
  __syncthreads();
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");   // this CTA runs and its tables are clear

  uint32_t key[kKpt];
  const float* xp = x + base;
  if (nv == kKpt && (reinterpret_cast<uintptr_t>(xp) & 15u) == 0u) {
#pragma unroll
    for (int e = 0; e < kKpt; e += 4) {
      const float4 v = __ldg(reinterpret_cast<const float4*>(xp + e));
      key[e] = order_key(v.x); key[e + 1] = order_key(v.y); key[e + 2] = order_key(v.z); key[e + 3] = order_key(v.w);
    }
  } else {
#pragma unroll
    for (int e = 0; e < kKpt; ++e) key[e] = e < nv ? order_key(__ldg(xp + e)) : 0u;
  }
#pragma unroll
  for (int e = 0; e < kKpt; ++e)
    if (e < nv) atomicAdd(&sm.hist[key[e] >> 21], 1u);
  __syncthreads();
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");     // every CTA of the cluster has done so

  uint32_t* peer_merged[kCluster];
#pragma unroll
  for (int p = 0; p < kCluster; ++p) peer_merged[p] = cluster.map_shared_rank(&sm.merged[0][0], p < n_cta ? p : 0);
  bool listed = false;

  for (int pass = 0; pass < 3; ++pass) {
    const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
    const uint32_t digit_mask = pass == 2 ? 1023u : 2047u;
    const uint32_t hi_mask = pass == 1 ? 0xffe00000u : 0xfffffc00u;
    const uint32_t prefix = sm.prefix;
    if (pass > 0) {
      if (listed) {
        const int n_cand = (int)sm.n_cand;
        for (int j = tid; j < n_cand; j += kTopkThreads) {
          const uint32_t c = sm.cand[j];
          if ((c & hi_mask) == prefix) atomicAdd(&sm.hist[(c >> shift) & digit_mask], 1u);
        }
      } else {
#pragma unroll
        for (int e = 0; e < kKpt; ++e)
          if (e < nv && (key[e] & hi_mask) == prefix) atomicAdd(&sm.hist[(key[e] >> shift) & digit_mask], 1u);
      }
      __syncthreads();
    }
    uint32_t local_bins[kBins / kTopkThreads];
    push_bins(sm, peer_merged, n_cta, pass, tid, local_bins);
    cluster.sync();
    select_digit(sm, pass, shift, prefix, tid, lane, warp);
    if (pass == 0) {
      const uint32_t digit0 = sm.prefix >> 21;
#pragma unroll
      for (int e = 0; e < kBins / kTopkThreads; ++e)
        if ((uint32_t)(tid + e * kTopkThreads) == digit0) sm.list_ok = local_bins[e] <= (uint32_t)kMaxCand;
      __syncthreads();
      listed = sm.list_ok != 0u;
      if (listed) {
#pragma unroll
        for (int e = 0; e < kKpt; ++e)
          if (e < nv && (key[e] >> 21) == digit0) sm.cand[atomicAdd(&sm.n_cand, 1u)] = key[e];
      }
      __syncthreads();
    }
  }

  const uint32_t thr = sm.prefix;          // key of the K-th largest score
  const uint32_t n_ties = sm.remaining;    // entries equal to it that are kept (lowest positions)

  // per thread: entries above the threshold (low half) and equal to it (high half; a CTA holds at most 16k keys)
  uint32_t mine = 0u;
#pragma unroll
  for (int e = 0; e < kKpt; ++e)
    if (e < nv) mine += (key[e] > thr ? 1u : 0u) + (key[e] == thr ? 0x10000u : 0u);
  uint32_t incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) sm.cnt_gt[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const uint32_t ws = sm.cnt_gt[lane];
    uint32_t wi = ws;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += y;
    }
    sm.cnt_eq[lane] = wi - ws;                             // packed counts of the warps before this one
    const uint32_t total = __shfl_sync(0xffffffffu, wi, 31);
    if (lane < n_cta) {                                    // lane p tells CTA p this CTA's totals
      *cluster.map_shared_rank(&sm.peer_gt[rank], lane) = total & 0xffffu;
      *cluster.map_shared_rank(&sm.peer_eq[rank], lane) = total >> 16;
    }
  }
  cluster.sync();                    // the last remote access of the kernel is behind every CTA
  uint32_t gt_before = 0u, eq_before = 0u;
  for (int r = 0; r < rank; ++r) { gt_before += sm.peer_gt[r]; eq_before += sm.peer_eq[r]; }
  const uint32_t before = sm.cnt_eq[warp] + (incl - mine);
  gt_before += before & 0xffffu;
  eq_before += before >> 16;
  uint32_t pos = gt_before + min(eq_before, n_ties);
#pragma unroll
  for (int e = 0; e < kKpt; ++e) {
    if (e < nv) {
      const bool eq = key[e] == thr;
      if (key[e] > thr || (eq && eq_before < n_ties)) out[pos++] = base + e;
      eq_before += eq ? 1u : 0u;
    }
  }
}

}  // namespace

cudaError_t launch_topk(const float* scores, int64_t score_stride, int32_t* idx, int64_t idx_stride,
                        const SeqTable& t, int n_kv_heads, cudaStream_t s, LaunchLog* log) {
  int max_len = 1;
  for (int b = 0; b < t.batch; ++b) max_len = t.prompt_len[b] > max_len ? t.prompt_len[b] : max_len;
  int n_cta = 1;
  while (n_cta < kCluster && (int64_t)n_cta * kKeysPerCta < max_len) n_cta *= 2;
  while (n_cta > 1 && t.batch * n_kv_heads * n_cta > kWaveCtas && (int64_t)(n_cta / 2) * 4 * kKeysPerCta >= max_len) n_cta /= 2;
  const int slice = (((max_len + n_cta - 1) / n_cta) + 31) & ~31;
  const dim3 grid(t.batch * n_cta, n_kv_heads), block(kTopkThreads);
  cudaError_t e;
  if (slice <= 16 * kTopkThreads) {                                   // keys in registers: 4, 8 or 16 per thread
    auto launch = [&](auto kernel) {
      cudaError_t le = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TopkSmem));
      if (le != cudaSuccess) return le;
      log->begin(kKindTopk, s);
      le = launch_pdl(kernel, grid, block, sizeof(TopkSmem), s, n_cta, scores, score_stride, idx, idx_stride, t);
      log->end(s);
      return le != cudaSuccess ? le : cudaGetLastError();
    };
    if (slice <= 4 * kTopkThreads) return launch(topk_select_reg_kernel<4>);
    if (slice <= 8 * kTopkThreads) return launch(topk_select_reg_kernel<8>);
    return launch(topk_select_reg_kernel<16>);
  }
  const int cache_keys = slice <= kMaxSliceSmem ? slice : 0;          // 0: every pass re-reads global memory
  const size_t smem = sizeof(TopkSmem) + (size_t)cache_keys * sizeof(uint32_t);
  e = cudaFuncSetAttribute(topk_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)(sizeof(TopkSmem) + (size_t)kMaxSliceSmem * sizeof(uint32_t)));
  if (e != cudaSuccess) return e;
  log->begin(kKindTopk, s);
  e = launch_pdl(topk_select_kernel, grid, block, smem, s, n_cta, scores, score_stride, idx, idx_stride, t, cache_keys);
  log->end(s);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace dapq
