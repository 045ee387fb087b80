// Per-head selection of the retained tokens (Section 4.2, Eq. 5: M_retain = TopK_j S(j)).
//
// One thread-block cluster of 1, 2, 4 or 8 CTAs (by the longest sequence: 4k to 32k keys per CTA, fewer CTAs
// when the grid would not fit one wave) per (sequence, KV head).  Each CTA owns a contiguous slice of the head's
// scores and reads it from global memory once.  A 3-pass radix select (11 + 11 + 10 bits of the scores'
// order-preserving integer images, most significant first) finds the exact bit pattern of the K-th largest
// score and how many entries equal to it still fit; an ordered compaction then writes, in ascending position,
// every entry above the threshold plus the lowest-position ties.  Integer work only: exact and deterministic.
//
// First pass, both kernels: every CTA histograms its slice with plain shared-memory atomics, adds its non-empty
// bins into the table of EVERY CTA of the cluster through distributed shared memory (remote adds need no
// reply), and after one cluster barrier scans its own copy of the merged table for the digit that holds the K-th
// entry.  No CTA ever reads remote memory, and none has to outlive another.
//   topk_select_reg_kernel (slices of up to 32k keys: sequences of up to 256k keys): keys in registers; after the
//     first pass the CTAs exchange the keys of the selected bin and finish by themselves (see the kernel).
//   topk_select_solo_kernel: the same with one CTA per head (short sequences, batches of sequences of up to 16k keys).
//   topk_select_kernel (longer slices): keys in shared memory or re-read from global memory; every pass merges
//     histograms across the cluster, and the CTAs push their totals to each other before the ordered write.
#include <cooperative_groups.h>

#include "dapq_internal.cuh"

namespace cg = cooperative_groups;

namespace dapq {
namespace {

constexpr int kTopkThreads = 1024;
constexpr int kWarps = kTopkThreads / 32;
constexpr int kCluster = 8;                   // most CTAs per (sequence, head); portable cluster size
constexpr int kKeysPerCta = 4096;             // general kernel: a CTA owns at least this many keys, up to four times as many
constexpr int kWaveCtas = 296;                // when the grid would otherwise exceed one wave (2 CTAs per SM)
constexpr int kBins = 2048;                   // 11-bit digits (the last pass uses 1024 of them)
constexpr int kMaxSliceSmem = 36864;          // keys a CTA can cache (144 KB); longer slices re-read global
constexpr int kMaxCand = 4096;                // candidate keys a CTA lists after the first pass (general kernel)
constexpr int kCap = 16384;                   // candidate keys of a whole cluster that the keys-in-registers kernel exchanges

// Monotone map float -> uint32 (larger float <=> larger key), valid for all finite values.
__device__ __forceinline__ uint32_t order_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct TopkTables {
  uint32_t merged[3][kBins];   // cluster-wide histogram of each pass (every CTA holds a copy)
  uint32_t hist[kBins];        // this CTA's histogram (all zero between passes)
  uint32_t warp_sum[kWarps];
  uint32_t cnt_gt[kWarps], cnt_eq[kWarps];
  uint32_t peer_gt[kCluster], peer_eq[kCluster];   // totals of every CTA of the cluster, pushed by their owners
  uint32_t prefix, remaining, n_cand, own_count, bin_total;
};

struct TopkSmem {              // general kernel; the cached keys follow
  TopkTables tb;
  uint32_t cand[kMaxCand];     // this CTA's keys that share the first pass's digit
};

struct TopkRegSmem {           // keys-in-registers kernel
  TopkTables tb;
  uint32_t cand[kCap];         // the candidates of EVERY CTA of the cluster: CTA r's block is [blk_base[r], + blk_cnt[r])
  uint32_t fill;               // slots of cand reserved so far (the CTAs of the cluster add their counts to it)
  uint32_t blk_base[kCluster], blk_cnt[kCluster];
  uint32_t my_base[kCluster];  // where this CTA's block starts in the list of CTA p
  uint32_t peer_hi[kCluster];  // how many keys of CTA r lie above the first pass's digit
  uint32_t reg_gt[kCluster], reg_eq[kCluster];
  uint32_t own_tally;          // this CTA's candidates listed so far (low half) and keys above the bin (high half)
};

// Thread t owns digits 2047-2t and 2046-2t of every table.  Adds this CTA's non-empty bins into the merged
// table of every CTA of the cluster and leaves the local table clear; local keeps the thread's own two counts.
__device__ __forceinline__ void push_bins(TopkTables& tb, cg::cluster_group& cluster, int n_cta, int pass, int tid,
                                          uint32_t (&local)[2]) {
  const int d_hi = kBins - 1 - 2 * tid;
  const uint2 c2 = *reinterpret_cast<const uint2*>(&tb.hist[d_hi - 1]);
  local[0] = c2.y;
  local[1] = c2.x;
  if (c2.x | c2.y) {
    *reinterpret_cast<uint2*>(&tb.hist[d_hi - 1]) = make_uint2(0u, 0u);
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      if (local[e]) {
        uint32_t* mine = &tb.merged[pass][d_hi - e];
        for (int p = 0; p < n_cta; ++p) atomicAdd(cluster.map_shared_rank(mine, p), local[e]);
      }
    }
  }
}

// Scans `table` from the top digit down for the digit that holds the entry of rank tb.remaining; extends
// tb.prefix by it, reduces tb.remaining to the rank within that digit and leaves this CTA's own count of the
// digit in tb.own_count and the table's in tb.bin_total.  Every warp sums the totals of the warps before it by itself: two block barriers.
__device__ __forceinline__ void select_digit(TopkTables& tb, const uint32_t* table, int shift, uint32_t prefix,
                                             const uint32_t (&local)[2], int tid, int lane, int warp) {
  const uint32_t remaining = tb.remaining;
  const int d_hi = kBins - 1 - 2 * tid;
  const uint2 v = *reinterpret_cast<const uint2*>(&table[d_hi - 1]);
  const uint32_t v0 = v.y, v1 = v.x;
  const uint32_t mine = v0 + v1;
  uint32_t incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) tb.warp_sum[warp] = incl;
  __syncthreads();
  uint32_t before = lane < warp ? tb.warp_sum[lane] : 0u;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
  incl += before;
  const uint32_t excl = incl - mine;
  if (excl < remaining && incl >= remaining) {           // exactly one thread
    const bool first = excl + v0 >= remaining;
    tb.prefix = prefix | ((uint32_t)(first ? d_hi : d_hi - 1) << shift);
    tb.remaining = remaining - excl - (first ? 0u : v0);
    tb.own_count = first ? local[0] : local[1];
    tb.bin_total = first ? v0 : v1;
  }
  __syncthreads();
}

// Block-wide exclusive prefix, in thread order, of `mine` (entries above the threshold in the low half, equal to
// it in the high half; a CTA holds at most 32k keys).  *total: the block's sum.  One block barrier.
__device__ __forceinline__ uint32_t packed_prefix(TopkTables& tb, uint32_t mine, int lane, int warp, uint32_t* total) {
  uint32_t incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) tb.cnt_gt[warp] = incl;
  __syncthreads();
  const uint32_t ws = tb.cnt_gt[lane];
  uint32_t before = lane < warp ? ws : 0u, all = ws;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    before += __shfl_xor_sync(0xffffffffu, before, o);
    all += __shfl_xor_sync(0xffffffffu, all, o);
  }
  *total = all;
  return before + incl - mine;
}

__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

__global__ void __launch_bounds__(kTopkThreads)
topk_select_kernel(const float* __restrict__ scores, int64_t score_stride, int32_t* __restrict__ idx,
                   int64_t idx_stride, const __grid_constant__ SeqTable t, int cache_keys) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  TopkSmem& sm = *reinterpret_cast<TopkSmem*>(smem_raw);
  TopkTables& tb = sm.tb;
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
  for (int d = tid; d < 3 * kBins; d += kTopkThreads) (&tb.merged[0][0])[d] = 0u;
  for (int d = tid; d < kBins; d += kTopkThreads) tb.hist[d] = 0u;
  if (tid == 0) { tb.prefix = 0u; tb.remaining = (uint32_t)K; tb.n_cand = 0u; }
  if (cached) {
    for (int j = tid; j < n_own; j += kTopkThreads) keys[j] = order_key(x[j0 + j]);
  }
  cluster.sync();                    // every CTA of the cluster runs and has cleared its tables

  bool listed = false;               // the later passes read the candidate list instead of the slice

  for (int pass = 0; pass < 3; ++pass) {
    const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
    const uint32_t digit_mask = pass == 2 ? 1023u : 2047u;
    const uint32_t hi_mask = pass == 0 ? 0u : (pass == 1 ? 0xffe00000u : 0xfffffc00u);
    const uint32_t prefix = tb.prefix;
    const int n_scan = listed ? (int)tb.n_cand : n_own;
    for (int j = tid; j < n_scan; j += kTopkThreads) {
      const uint32_t key = listed ? sm.cand[j] : (cached ? keys[j] : order_key(x[j0 + j]));
      if ((key & hi_mask) == prefix) atomicAdd(&tb.hist[(key >> shift) & digit_mask], 1u);
    }
    __syncthreads();
    uint32_t local[2];
    push_bins(tb, cluster, n_cta, pass, tid, local);
    cluster.sync();
    select_digit(tb, tb.merged[pass], shift, prefix, local, tid, lane, warp);
    if (pass == 0) {
      // keep only this CTA's keys of the selected bin, if they fit the list
      const uint32_t digit0 = tb.prefix >> 21;
      listed = tb.own_count <= (uint32_t)kMaxCand;
      if (listed) {
        for (int j = tid; j < n_own; j += kTopkThreads) {
          const uint32_t key = cached ? keys[j] : order_key(x[j0 + j]);
          if ((key >> 21) == digit0) sm.cand[atomicAdd(&tb.n_cand, 1u)] = key;
        }
      }
      __syncthreads();
    }
  }

  const uint32_t thr = tb.prefix;          // key of the K-th largest score
  const uint32_t n_ties = tb.remaining;    // entries equal to it that are kept (lowest positions)

  // ordered compaction: within the CTA, warp w owns the contiguous span [w * span, (w+1) * span)
  const int span = (((n_own + kWarps - 1) / kWarps) + 31) & ~31;
  const int s0 = min(n_own, warp * span), s1 = min(n_own, s0 + span);
  uint32_t n_gt = 0u, n_eq = 0u;
  for (int j = s0 + lane; j < s0 + span; j += 32) {
    const uint32_t key = (j < s1) ? (cached ? keys[j] : order_key(x[j0 + j])) : 0u;
    n_gt += __popc(__ballot_sync(0xffffffffu, j < s1 && key > thr));
    n_eq += __popc(__ballot_sync(0xffffffffu, j < s1 && key == thr));
  }
  if (lane == 0) { tb.cnt_gt[warp] = n_gt; tb.cnt_eq[warp] = n_eq; }
  __syncthreads();
  if (warp == 0) {
    uint32_t g = tb.cnt_gt[lane], e = tb.cnt_eq[lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      g += __shfl_xor_sync(0xffffffffu, g, o);
      e += __shfl_xor_sync(0xffffffffu, e, o);
    }
    if (lane < n_cta) {                                    // lane p tells CTA p this CTA's totals
      *cluster.map_shared_rank(&tb.peer_gt[rank], lane) = g;
      *cluster.map_shared_rank(&tb.peer_eq[rank], lane) = e;
    }
  }
  cluster.sync();                    // the last remote access of the kernel is behind every CTA
  uint32_t gt_before = 0u, eq_before = 0u;
  for (int r = 0; r < rank; ++r) { gt_before += tb.peer_gt[r]; eq_before += tb.peer_eq[r]; }
  for (int w = 0; w < warp; ++w) { gt_before += tb.cnt_gt[w]; eq_before += tb.cnt_eq[w]; }
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

// The same selection for slices of up to 16k keys per CTA (sequences of up to 128k keys).  Thread t of CTA r owns
// the kKpt CONSECUTIVE keys from position (r * 1024 + t) * kKpt and holds them in registers: every scan is an
// unrolled register loop, and the final order (ascending position) is the thread order, so one block-wide prefix
// sum of the threads' counts places every kept entry.  Everything that does not depend on the scores (tables,
// the first cluster barrier's arrival) runs before the wait for the kernel that writes them.  After the first
// pass every CTA sends its candidates (the keys of the selected bin) and its count of the keys above that bin to
// ALL CTAs of the cluster; if every CTA's candidates fit their region, each CTA finishes the selection by itself
// on its copy of the candidates and derives the other CTAs' totals from them: two cluster barriers in all, none
// after the exchange, so no CTA waits for another at the end.  Otherwise (a bin that holds thousands of a CTA's
// keys) the later passes merge histograms across the cluster like the general kernel.
template <int kKpt, int kMinCtas>
__global__ void __launch_bounds__(kTopkThreads, kMinCtas)
topk_select_reg_kernel(const float* __restrict__ scores, int64_t score_stride, int32_t* __restrict__ idx,
                       int64_t idx_stride, const __grid_constant__ SeqTable t) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  TopkRegSmem& sm = *reinterpret_cast<TopkRegSmem*>(smem_raw);
  TopkTables& tb = sm.tb;

  pdl_trigger();
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

  for (int d = tid; d < 3 * kBins; d += kTopkThreads) (&tb.merged[0][0])[d] = 0u;
  for (int d = tid; d < kBins; d += kTopkThreads) tb.hist[d] = 0u;
  if (tid == 0) { tb.prefix = 0u; tb.remaining = (uint32_t)K; sm.fill = 0u; sm.own_tally = 0u; }
  if (tid < kCluster) { sm.reg_gt[tid] = 0u; sm.reg_eq[tid] = 0u; }
  __syncthreads();
  cluster_arrive();                  // this CTA runs and its tables are clear
  pdl_wait();                        // the scores are written, and the index buffer's last reader is done

  if (K >= L) {                      // keep everything (uniform over the cluster)
    cluster_wait();
    for (int e = 0; e < nv; ++e) out[base + e] = base + e;
    return;
  }

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
    if (e < nv) atomicAdd(&tb.hist[key[e] >> 21], 1u);
  __syncthreads();
  cluster_wait();                    // every CTA of the cluster has arrived: remote adds may start

  uint32_t local[2];
  push_bins(tb, cluster, n_cta, 0, tid, local);
  cluster.sync();
  select_digit(tb, tb.merged[0], 21, 0u, local, tid, lane, warp);

  // If the selected bin's keys (the candidates) fit one list, every CTA sends its own, and its count of the keys
  // above the bin, to ALL CTAs of the cluster.  The bin's cluster-wide count is the same in every CTA's table:
  // the whole cluster takes one branch.
  const uint32_t digit0 = tb.prefix >> 21;
  const uint32_t own = tb.own_count;
  const bool all_fit = tb.bin_total <= (uint32_t)kCap;
  uint32_t gt_before = 0u, eq_before = 0u;   // of the CTAs before this one
  if (all_fit) {
    if (tid < n_cta) {               // thread p reserves this CTA's block in the list of CTA p and tells it where the block lies
      const uint32_t at = atomicAdd(cluster.map_shared_rank(&sm.fill, tid), own);
      sm.my_base[tid] = at;
      *cluster.map_shared_rank(&sm.blk_base[rank], tid) = at;
      *cluster.map_shared_rank(&sm.blk_cnt[rank], tid) = own;
    }
    uint32_t tally = 0u;             // candidates (low half) and keys above the bin (high half) of this thread
#pragma unroll
    for (int e = 0; e < kKpt; ++e) {
      if (e < nv) {
        const uint32_t d = key[e] >> 21;
        tally += (d == digit0 ? 1u : 0u) + (d > digit0 ? 0x10000u : 0u);
      }
    }
    uint32_t incl = tally;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    uint32_t warp_at = 0u;
    if (lane == 31 && incl) warp_at = atomicAdd(&sm.own_tally, incl);
    warp_at = __shfl_sync(0xffffffffu, warp_at, 31);
    __syncthreads();                 // the block starts are known
    uint32_t at = sm.my_base[rank] + ((warp_at + incl - tally) & 0xffffu);
#pragma unroll
    for (int e = 0; e < kKpt; ++e)
      if (e < nv && (key[e] >> 21) == digit0) sm.cand[at++] = key[e];
    __syncthreads();
    {
      const uint32_t from = sm.my_base[rank];
      for (int j = tid; j < (int)own; j += kTopkThreads) {
        const uint32_t c = sm.cand[from + j];
        for (int p = 0; p < n_cta; ++p)
          if (p != rank) *cluster.map_shared_rank(&sm.cand[sm.my_base[p] + j], p) = c;
      }
    }
    if (tid < n_cta) *cluster.map_shared_rank(&sm.peer_hi[rank], tid) = sm.own_tally >> 16;
    cluster.sync();                  // the last remote access of this branch is behind every CTA

    // passes 2 and 3 on this CTA's copy of all candidates (tables 1 and 2 serve as local histograms)
    const int n_all = (int)tb.bin_total;
    for (int pass = 1; pass < 3; ++pass) {
      const int shift = pass == 1 ? 10 : 0;
      const uint32_t digit_mask = pass == 2 ? 1023u : 2047u;
      const uint32_t hi_mask = pass == 1 ? 0xffe00000u : 0xfffffc00u;
      const uint32_t prefix = tb.prefix;
      for (int j = tid; j < n_all; j += kTopkThreads) {
        const uint32_t c = sm.cand[j];
        if ((c & hi_mask) == prefix) atomicAdd(&tb.merged[pass][(c >> shift) & digit_mask], 1u);
      }
      __syncthreads();
      select_digit(tb, tb.merged[pass], shift, prefix, local, tid, lane, warp);
    }
    const uint32_t thr = tb.prefix;
    {                                // warps r, r + n_cta, ... share the block of CTA r: its entries above / equal to the threshold
      const int r = warp % n_cta, from = (int)sm.blk_base[r], n = (int)sm.blk_cnt[r];
      uint32_t g = 0u, q = 0u;
      for (int j = (warp / n_cta) * 32 + lane; j < n; j += 32 * (kWarps / n_cta)) {
        const uint32_t c = sm.cand[from + j];
        g += c > thr ? 1u : 0u;
        q += c == thr ? 1u : 0u;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        g += __shfl_xor_sync(0xffffffffu, g, o);
        q += __shfl_xor_sync(0xffffffffu, q, o);
      }
      if (lane == 0) {
        if (g) atomicAdd(&sm.reg_gt[r], g);
        if (q) atomicAdd(&sm.reg_eq[r], q);
      }
    }
  } else {
    for (int pass = 1; pass < 3; ++pass) {
      const int shift = pass == 1 ? 10 : 0;
      const uint32_t digit_mask = pass == 2 ? 1023u : 2047u;
      const uint32_t hi_mask = pass == 1 ? 0xffe00000u : 0xfffffc00u;
      const uint32_t prefix = tb.prefix;
#pragma unroll
      for (int e = 0; e < kKpt; ++e)
        if (e < nv && (key[e] & hi_mask) == prefix) atomicAdd(&tb.hist[(key[e] >> shift) & digit_mask], 1u);
      __syncthreads();
      push_bins(tb, cluster, n_cta, pass, tid, local);
      cluster.sync();
      select_digit(tb, tb.merged[pass], shift, prefix, local, tid, lane, warp);
    }
  }

  const uint32_t thr = tb.prefix;          // key of the K-th largest score
  const uint32_t n_ties = tb.remaining;    // entries equal to it that are kept (lowest positions)
  uint32_t mine = 0u;
#pragma unroll
  for (int e = 0; e < kKpt; ++e)
    if (e < nv) mine += (key[e] > thr ? 1u : 0u) + (key[e] == thr ? 0x10000u : 0u);
  uint32_t total;
  const uint32_t before = packed_prefix(tb, mine, lane, warp, &total);   // (its barrier also publishes reg_gt / reg_eq)
  if (all_fit) {
    for (int r = 0; r < rank; ++r) { gt_before += sm.reg_gt[r] + sm.peer_hi[r]; eq_before += sm.reg_eq[r]; }
  } else {
    if (tid < n_cta) {                                     // thread p tells CTA p this CTA's totals
      *cluster.map_shared_rank(&tb.peer_gt[rank], tid) = total & 0xffffu;
      *cluster.map_shared_rank(&tb.peer_eq[rank], tid) = total >> 16;
    }
    cluster.sync();                  // the last remote access of the kernel is behind every CTA
    for (int r = 0; r < rank; ++r) { gt_before += tb.peer_gt[r]; eq_before += tb.peer_eq[r]; }
  }
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

// One CTA per (sequence, KV head), for sequences of up to 16k keys when a cluster per head would not fit one wave
// (batches): the same steps as topk_select_reg_kernel without any exchange: the three tables are local histograms.
template <int kKpt>
__global__ void __launch_bounds__(kTopkThreads)
topk_select_solo_kernel(const float* __restrict__ scores, int64_t score_stride, int32_t* __restrict__ idx,
                        int64_t idx_stride, const __grid_constant__ SeqTable t) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  TopkRegSmem& sm = *reinterpret_cast<TopkRegSmem*>(smem_raw);
  TopkTables& tb = sm.tb;

  pdl_trigger();
  const int b = blockIdx.x, kvh = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int L = t.prompt_len[b];
  const int K = t.cu_keep[b + 1] - t.cu_keep[b];
  const float* x = scores + (int64_t)kvh * score_stride + t.cu_prompt[b];
  int32_t* out = idx + (int64_t)kvh * idx_stride + t.cu_keep[b];
  const int base = tid * kKpt;
  const int nv = max(0, min(kKpt, L - base));

  for (int d = tid; d < 3 * kBins; d += kTopkThreads) (&tb.merged[0][0])[d] = 0u;
  if (tid == 0) { tb.prefix = 0u; tb.remaining = (uint32_t)K; sm.own_tally = 0u; }
  __syncthreads();
  pdl_wait();                        // the scores are written, and the index buffer's last reader is done

  if (K >= L) {
    for (int e = 0; e < nv; ++e) out[base + e] = base + e;
    return;
  }

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
    if (e < nv) atomicAdd(&tb.merged[0][key[e] >> 21], 1u);
  __syncthreads();
  const uint32_t local[2] = {0u, 0u};
  select_digit(tb, tb.merged[0], 21, 0u, local, tid, lane, warp);

  // the selected bin's keys (the candidates) go to the list (a CTA's keys always fit it); the later passes read it
  static_assert(kKpt * kTopkThreads <= kCap, "one CTA's keys must fit the candidate list");
  const uint32_t digit0 = tb.prefix >> 21;
  const int n_all = (int)tb.bin_total;
  {
    uint32_t mine = 0u;
#pragma unroll
    for (int e = 0; e < kKpt; ++e)
      if (e < nv && (key[e] >> 21) == digit0) ++mine;
    uint32_t incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    uint32_t warp_at = 0u;
    if (lane == 31 && incl) warp_at = atomicAdd(&sm.own_tally, incl);
    uint32_t at = __shfl_sync(0xffffffffu, warp_at, 31) + incl - mine;
#pragma unroll
    for (int e = 0; e < kKpt; ++e)
      if (e < nv && (key[e] >> 21) == digit0) sm.cand[at++] = key[e];
    __syncthreads();
  }
  for (int pass = 1; pass < 3; ++pass) {
    const int shift = pass == 1 ? 10 : 0;
    const uint32_t digit_mask = pass == 2 ? 1023u : 2047u;
    const uint32_t hi_mask = pass == 1 ? 0xffe00000u : 0xfffffc00u;
    const uint32_t prefix = tb.prefix;
    for (int j = tid; j < n_all; j += kTopkThreads) {
      const uint32_t c = sm.cand[j];
      if ((c & hi_mask) == prefix) atomicAdd(&tb.merged[pass][(c >> shift) & digit_mask], 1u);
    }
    __syncthreads();
    select_digit(tb, tb.merged[pass], shift, prefix, local, tid, lane, warp);
  }

  const uint32_t thr = tb.prefix;          // key of the K-th largest score
  const uint32_t n_ties = tb.remaining;    // entries equal to it that are kept (lowest positions)
  uint32_t mine = 0u;
#pragma unroll
  for (int e = 0; e < kKpt; ++e)
    if (e < nv) mine += (key[e] > thr ? 1u : 0u) + (key[e] == thr ? 0x10000u : 0u);
  uint32_t total;
  const uint32_t before = packed_prefix(tb, mine, lane, warp, &total);
  uint32_t eq_before = before >> 16;
  uint32_t pos = (before & 0xffffu) + min(eq_before, n_ties);
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

namespace {

// Cluster size, keys per thread and CTAs per SM of the keys-in-registers kernels for `heads` (sequence, head)
// problems of up to max_len keys: the cheapest by a small model of their run time (waves of CTAs, a fixed part per
// CTA that is larger with a cluster, a part per key of a thread).  Instances of up to 16 keys per thread fit two
// CTAs on an SM.  n_cta = 0: the slices are too long for registers.
struct TopkShape { int n_cta, kpt, per_sm; };

TopkShape plan_topk(int heads, int max_len, int n_sm) {
  TopkShape best = {0, 0, 1};
  double best_cost = 0.0;
  for (int n_cta = 1; n_cta <= kCluster; n_cta *= 2) {
    const int slice = (max_len + n_cta - 1) / n_cta;
    if (slice > 32 * kTopkThreads) continue;
    const int kpt = slice <= 4 * kTopkThreads ? 4 : (slice <= 8 * kTopkThreads ? 8 : (slice <= 16 * kTopkThreads ? 16 : 32));
    if (n_cta == 1 && kpt == 32) continue;              // (a cluster of two with 16 keys per thread is never slower)
    const int ctas = heads * n_cta;
    const int per_sm = (kpt <= 16 && ctas > n_sm) ? 2 : 1;
    const int waves = (ctas + n_sm * per_sm - 1) / (n_sm * per_sm);
    const double cost = waves * ((n_cta == 1 ? 5.0 : 7.0) + 0.2 * kpt);
    if (best.n_cta == 0 || cost < best_cost) { best = {n_cta, kpt, per_sm}; best_cost = cost; }
  }
  return best;
}

}  // namespace

cudaError_t launch_topk(const float* scores, int64_t score_stride, int32_t* idx, int64_t idx_stride,
                        const SeqTable& t, int n_kv_heads, cudaStream_t s, LaunchLog* log) {
  int max_len = 1;
  for (int b = 0; b < t.batch; ++b) max_len = t.prompt_len[b] > max_len ? t.prompt_len[b] : max_len;
  int dev = 0, n_sm = 148;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  const TopkShape shape = plan_topk(t.batch * n_kv_heads, max_len, n_sm);
  if (shape.n_cta > 0) {                                              // keys in registers: 4, 8, 16 or 32 per thread
    const int n_cta = shape.n_cta;
    const dim3 grid(t.batch * n_cta, n_kv_heads), block(kTopkThreads);
    auto launch = [&](auto kernel) {
      cudaError_t le = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TopkRegSmem));
      if (le != cudaSuccess) return le;
      log->begin(kKindTopk, s);
      le = launch_pdl(kernel, grid, block, sizeof(TopkRegSmem), s, n_cta, scores, score_stride, idx, idx_stride, t);
      log->end(s);
      return le != cudaSuccess ? le : cudaGetLastError();
    };
    const bool two = shape.per_sm == 2;
    if (n_cta == 1) {
      switch (shape.kpt) {
        case 4: return launch(topk_select_solo_kernel<4>);
        case 8: return launch(topk_select_solo_kernel<8>);
        default: return launch(topk_select_solo_kernel<16>);
      }
    }
    switch (shape.kpt) {
      case 4: return two ? launch(topk_select_reg_kernel<4, 2>) : launch(topk_select_reg_kernel<4, 1>);
      case 8: return two ? launch(topk_select_reg_kernel<8, 2>) : launch(topk_select_reg_kernel<8, 1>);
      case 16: return two ? launch(topk_select_reg_kernel<16, 2>) : launch(topk_select_reg_kernel<16, 1>);
      default: return launch(topk_select_reg_kernel<32, 1>);
    }
  }
  int n_cta = kCluster;
  while (n_cta > 1 && t.batch * n_kv_heads * n_cta > kWaveCtas && (int64_t)(n_cta / 2) * 4 * kKeysPerCta >= max_len) n_cta /= 2;
  const int slice = (((max_len + n_cta - 1) / n_cta) + 31) & ~31;
  const dim3 grid(t.batch * n_cta, n_kv_heads), block(kTopkThreads);
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
