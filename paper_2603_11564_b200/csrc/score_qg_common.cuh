// Definitions shared by the two sweeps of the tensor-core scorer in its one-query-group-per-CTA
// form (see score_qg.cu): geometry, shared-memory layout, barriers, and the roles that feed the MMAs.
#pragma once
#include <cuda_fp16.h>

#include "umma_ptx.cuh"

namespace dapq {
namespace qg {

using namespace ptx;

constexpr int kTile1 = 192;                    // keys per K tile of sweep 1 (= UMMA N there)
constexpr int kTile2 = 128;                    // keys per K tile of sweep 2 (= UMMA M there)
constexpr int kGroupRows = 256;                // most query rows a CTA keeps resident
constexpr int kEpiGroups = 4;                  // epilogue groups of 4 warps (128 TMEM lanes each)
constexpr int kConvWarps = 4;                  // warps that convert the K tiles in place
constexpr int kFirstEpiWarp = 2 + kConvWarps;
constexpr int kEpiThreads = kEpiGroups * 128;
constexpr int kThreads1 = (kFirstEpiWarp + 4 * kEpiGroups) * 32;        // sweep 1: 22 warps
constexpr int kThreads2 = kThreads1 + 32;                               // sweep 2: one more warp sums the groups' partials
constexpr int kTmemCols = 512;
constexpr int kMaxStages = 4, kMaxAcc = 4;
constexpr int kExchDepth = 4;                  // jobs whose partial sums can wait in shared memory (sweep 2)
constexpr int kWideRows = 2 * kGroupRows;      // ... in the wide form of sweep 2 (two accumulators' worth of query columns)
// Sweep 2 with its own fp16 queries appends one k-step to every job's MMAs that adds -lse_i to column i of
// the accumulator: a [rows x 16] operand holding -lse as an fp16 pair, against a [128 x 16] operand of ones.
// Sweep 1 does the same with a per-row reference logit (its [256 x 16] operand also sits at the end of the
// ring area; its [192 x 16] operand of ones takes the place of sweep 2's exchange ring behind the barriers).
constexpr int kOnesSlabBytes = kTile2 * 32, kOnes1SlabBytes = kTile1 * 32;

template <int kTile>
struct TileGeo {
  static constexpr int kStage = kTile * 256;   // one K tile: two 64-channel halves of kTile rows x 128 B
  static constexpr int kHalf = kTile * 128;
};

// Shared memory (offsets from the 1024-aligned base): queries, K ring and the extra operands up to ring_end,
// the small state behind it.  kWide: room for 512 query rows (sweep 2 only).
template <bool kWide>
struct SmemT {
  static constexpr int rows = kWide ? kWideRows : kGroupRows;
  static constexpr int ring_end = (kWide ? 214 : 216) * 1024;
  static constexpr int lse_slab_bytes = rows * 32, slab_bytes = lse_slab_bytes + kOnesSlabBytes;
  static constexpr int lse_slab = ring_end - slab_bytes, ones_slab = ring_end - kOnesSlabBytes;   // sweep 2's extra operands
  static constexpr int ref_slab_bytes = rows * 32, ref_slab = ring_end - ref_slab_bytes;          // sweep 1's
  static constexpr int bars = ring_end;
  // barriers: k_full[4], k_conv[4], k_empty[4], acc_full[4], acc_empty[4], part_full[4], part_empty[4], q_full, drain, lse_ready
  static constexpr int n_bars = 3 * kMaxStages + 2 * kMaxAcc + 2 * kExchDepth + 3;
  static constexpr int lse = (bars + n_bars * 8 + 15) & ~15;       // [rows] floats, read as float4 (sweep 2); with the next block:
                                                                   // [rows] float2 row statistics (sweep 1)
  static constexpr int aux = lse + rows * 4;                       // [rows] floats: the other half of the statistics
  static constexpr int exch = aux + rows * 4;                      // [kExchDepth][4][128] floats (sweep 2)
  static constexpr int tmem_ptr = exch + kExchDepth * kEpiGroups * 128 * 4;
  static constexpr int abort_flag = tmem_ptr + 4;
  static constexpr int total = abort_flag + 4;
  static_assert(lse % 16 == 0 && aux % 16 == 0 && exch % 256 == 0, "vector loads need 16-byte alignment, MMA operands 256");
  static_assert(total <= 232448, "exceeds the shared memory a CTA can opt in to");
};
using Smem = SmemT<false>;
constexpr int kRingEnd = Smem::ring_end;
constexpr int kLseSlabBytes = Smem::lse_slab_bytes, kSlabBytes = Smem::slab_bytes;
constexpr int kLseSlab = Smem::lse_slab, kOnesSlab = Smem::ones_slab;
constexpr int kRefSlabBytes = Smem::ref_slab_bytes, kRefSlab = Smem::ref_slab;
static_assert(kOnes1SlabBytes <= kExchDepth * kEpiGroups * 128 * 4, "sweep 1's operand of ones does not fit the exchange area");
constexpr int kSmemBytes = Smem::total;

struct Args {
  int32_t n_pseudo, group, n_q_heads, n_kv_heads;
  int32_t rows_total;        // G * N query rows per KV head
  int32_t n_qgroups;         // CTAs that share a K chunk, one query group each
  int32_t rows_g;            // rows per group (a multiple of 16; the last group may hold fewer)
  int32_t rows_pad;          // row pitch of `part`
  int32_t n_stages;          // K stages that fit beside the group's queries
  int32_t early_loads;       // the kernel before this one in the stream is one of this library's that waited for ITS
                             // predecessor: inputs it does not write may be copied before this kernel's own wait
  float scale_log2e;
  long long wait_limit;      // cycles a wait may take before the CTA gives up
  float2* part;              // [n_chunks1, H_kv, rows_pad] (running max, sum) of every query row over a chunk's keys, base 2
  const float* ref;          // [B, H_q, N] base-2 reference logit of every query row (fp16 queries only)
  const float* lse_in;       // [B, H_q, N] natural-log lse from the caller, or NULL (use part)
  float* lse_out;            // [B, H_q, N] natural-log lse used, or NULL
  float* scores;             // [n_qgroups][H_kv][score_stride] when n_qgroups > 1 (one slot per group), else [H_kv][score_stride]
  int64_t score_stride, slot_stride;
  int* status;
};

// This CTA's work: sequence, tile range, first cache row, its query group.
struct Work {
  int chunk, qgrp, b, L, nt, t0, row_base, qrow_base, rows, mb;
};
__device__ __forceinline__ Work cta_work(const SeqTable& t, const ChunkTable& ct, const Args& a, int tile_keys,
                                         bool with_synthetic) {
  Work w;
  w.chunk = blockIdx.x / a.n_qgroups;
  w.qgrp = blockIdx.x - w.chunk * a.n_qgroups;
  const int kvh = blockIdx.y;
  w.b = find_segment(ct.cu_chunk, t.batch, w.chunk);
  w.L = t.prompt_len[w.b];
  const int n_keys = w.L + (with_synthetic ? a.n_pseudo : 0);
  const int n_tiles = (n_keys + tile_keys - 1) / tile_keys;
  w.t0 = (w.chunk - ct.cu_chunk[w.b]) * ct.chunk_tiles;
  w.nt = min(n_tiles, w.t0 + ct.chunk_tiles) - w.t0;
  w.row_base = t.cu_rows[w.b];                                                    // first cache row of the sequence
  w.qrow_base = (w.b * a.n_q_heads + kvh * a.group) * a.n_pseudo;                 // first query row of this KV head
  w.rows = min(a.rows_g, a.rows_total - w.qgrp * a.rows_g);                       // query rows of this CTA's group
  w.mb = (w.rows + 127) / 128;                                                    // blocks of 128 rows
  return w;
}

struct Bars {
  uint32_t base;
  __device__ __forceinline__ uint32_t k_full(int s) const { return base + 8u * s; }
  __device__ __forceinline__ uint32_t k_conv(int s) const { return base + 8u * (kMaxStages + s); }
  __device__ __forceinline__ uint32_t k_empty(int s) const { return base + 8u * (2 * kMaxStages + s); }
  __device__ __forceinline__ uint32_t acc_full(int i) const { return base + 8u * (3 * kMaxStages + i); }
  __device__ __forceinline__ uint32_t acc_empty(int i) const { return base + 8u * (3 * kMaxStages + kMaxAcc + i); }
  __device__ __forceinline__ uint32_t part_full(int i) const { return base + 8u * (3 * kMaxStages + 2 * kMaxAcc + i); }
  __device__ __forceinline__ uint32_t part_empty(int i) const {
    return base + 8u * (3 * kMaxStages + 2 * kMaxAcc + kExchDepth + i);
  }
  __device__ __forceinline__ uint32_t q_full() const { return base + 8u * (3 * kMaxStages + 2 * kMaxAcc + 2 * kExchDepth); }
  __device__ __forceinline__ uint32_t drain() const { return base + 8u * (3 * kMaxStages + 2 * kMaxAcc + 2 * kExchDepth + 1); }
  __device__ __forceinline__ uint32_t lse_ready() const { return base + 8u * (3 * kMaxStages + 2 * kMaxAcc + 2 * kExchDepth + 2); }
};

// Position in a ring of n slots walked once per tile or job: slot index and the parity of its phase.
struct Ring {
  int n, i = 0;
  uint32_t phase = 0;
  bool wrapped = false;
  __device__ __forceinline__ explicit Ring(int n_) : n(n_) {}
  __device__ __forceinline__ void next() {
    if (++i == n) { i = 0; phase ^= 1u; wrapped = true; }
  }
};

// What a role needs to wait on a barrier: the CTA's abort flag, the status word, the cycle limit.
struct Waiter {
  volatile int* abort_flag;
  int* status;
  long long limit;
  __device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity) const {
    return mbar_wait_limit(bar, parity, abort_flag, status, limit);
  }
  __device__ __forceinline__ bool aborting() const { return *abort_flag != 0; }
};

// Arrivals that complete a phase of barrier `idx` (in the order of Bars).
__device__ __forceinline__ uint32_t bar_count(int idx) {
  if (idx < kMaxStages) return 1u;                                        // k_full: the producer (+ the copies' bytes)
  if (idx < 2 * kMaxStages) return kConvWarps;                            // k_conv
  if (idx < 3 * kMaxStages + kMaxAcc) return 1u;                          // k_empty, acc_full: one tcgen05.commit
  if (idx < 3 * kMaxStages + 2 * kMaxAcc + kExchDepth) return 4u * kEpiGroups;   // acc_empty, part_full: every epilogue warp
  return 1u;                                                              // part_empty, q_full, drain, lse_ready
}

// Common CTA prologue: barrier init (warp 0, one barrier per lane), the first TMA copies (`first`, run by
// thread 0 as soon as the barriers exist: only copies of data that the kernel before this one does not
// write), tensor-memory allocation (warp 1), one CTA-wide sync, then the wait for the kernel before this one
// (all of this overlaps that kernel's tail).  Returns the tensor-memory base address.
template <class Smem = SmemT<false>, class First>
__device__ __forceinline__ uint32_t cta_prologue(uint8_t* smem, uint32_t sbase, const Bars& bars, First first) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  static_assert(Smem::n_bars <= 32, "one barrier per lane of warp 0");
  if (warp == 0) {
    if (lane < Smem::n_bars) mbar_init(bars.base + 8u * lane, bar_count(lane));
    if (lane == 0) *reinterpret_cast<volatile int*>(smem + Smem::abort_flag) = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncwarp();
    if (lane == 0) first();
  }
  if (warp == 1) {                                              // tensor memory: all 512 columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(sbase + Smem::tmem_ptr), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();                                                   // what the previous kernel wrote is read only from here on
  return *reinterpret_cast<volatile uint32_t*>(smem + Smem::tmem_ptr);
}

__device__ __forceinline__ void cta_epilogue(uint32_t tmem_base) {
  tc_fence_before();
  __syncthreads();
  if ((threadIdx.x >> 5) == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ---- TMA producer (one thread).  tma_first issues the first K tile and, if the queries are not written by
// the kernel before this one (kWithQ), the CTA's query group; it runs inside the prologue.  tma_producer
// then issues the queries if they are still owed and the rest of the ring.  It returns only when every copy
// has landed (also when the CTA is aborting), so that the CTA never exits with a copy into its shared
// memory in flight.
__device__ __forceinline__ void tma_queries(const CUtensorMap* tm_q, const Work& w, const Args& a, uint32_t sbase, const Bars& bars) {
  const uint32_t q_bytes = (uint32_t)w.mb * 2u * 128u * 128u;
  mbar_expect_tx(bars.q_full(), q_bytes);
  for (int half = 0; half < 2; ++half)
    for (int m = 0; m < w.mb; ++m)
      tma_load_2d(sbase + half * (q_bytes / 2) + m * 128 * 128, tm_q, bars.q_full(), half * 64,
                  w.qrow_base + w.qgrp * a.rows_g + m * 128);
}
template <int kTile, bool kWithQ>
__device__ __forceinline__ void tma_first(const CUtensorMap* tm_k, const CUtensorMap* tm_q, const Work& w, const Args& a,
                                          uint32_t sbase, const Bars& bars, int kvh) {
  using T = TileGeo<kTile>;
  const uint32_t ring = sbase + (uint32_t)w.mb * 2u * 128u * 128u;
  mbar_expect_tx(bars.k_full(0), T::kStage);                // (w.nt >= 1: checked by the caller)
  const int row = w.row_base + w.t0 * kTile;
  tma_load_3d(ring, tm_k, bars.k_full(0), 0, row, kvh);
  tma_load_3d(ring + T::kHalf, tm_k, bars.k_full(0), 64, row, kvh);
  if (kWithQ) tma_queries(tm_q, w, a, sbase, bars);
}
// kQOwed: the queries were not part of tma_first.  kGate (sweep 2): the tiles after the first wait until the
// epilogue warps have merged sweep 1's partials: at the start of a launch every SM asks for its whole ring at
// once, and whatever is queued behind those copies takes microseconds to arrive.
template <int kTile, bool kQOwed, bool kGate>
__device__ __forceinline__ void tma_producer(const CUtensorMap* tm_k, const CUtensorMap* tm_q, const Work& w, const Args& a,
                                             uint32_t sbase, const Bars& bars, int kvh, const Waiter& wt) {
  using T = TileGeo<kTile>;
  const int S = a.n_stages;
  const uint32_t q_bytes = (uint32_t)w.mb * 2u * 128u * 128u;
  const uint32_t ring = sbase + q_bytes;
  int li = 1;                                               // K tiles issued so far (the first by tma_first)
  bool ok = true;
  auto load_tile = [&](int ti) {
    const int s = li % S;                                   // (li == ti; one division per tile in this single thread)
    mbar_expect_tx(bars.k_full(s), T::kStage);
    const int row = w.row_base + (w.t0 + ti) * kTile;
    tma_load_3d(ring + s * T::kStage, tm_k, bars.k_full(s), 0, row, kvh);
    tma_load_3d(ring + s * T::kStage + T::kHalf, tm_k, bars.k_full(s), 64, row, kvh);
    ++li;
  };
  if (kQOwed) {
    // (the first job needs the queries, not the tiles after the first: those go out once the queries are in)
    tma_queries(tm_q, w, a, sbase, bars);
    ok = wt.wait(bars.q_full(), 0);
  }
  if (kGate) ok = wt.wait(bars.lse_ready(), 0);
  Ring rs(S);
  for (int ti = 1; ti < w.nt && ok; ++ti) {
    rs.next();
    if (rs.wrapped) ok = wt.wait(bars.k_empty(rs.i), rs.phase ^ 1u);
    if (ok) load_tile(ti);
  }
  // See every copy issued above land before this thread (and with it the CTA) returns: in a normal run
  // they have all been consumed by now; in an aborting CTA nobody else may be left to wait for them.
  for (int back = 1; back <= S && back <= li; ++back) {
    const int l2 = li - back;
    drain_wait(bars.k_full(l2 % S), (l2 / S) & 1, kWaitLimit);
  }
  drain_wait(bars.q_full(), 0, kWaitLimit);
}

// ---- K tiles from bf16 to fp16, in place (kConvWarps warps).  bf16 -> fp16 keeps every value of
// magnitude 2^-14 .. 65504 exactly (8 significant bits fit 11); smaller ones round to multiples of
// 2^-24, larger ones saturate.  The element size does not change, so neither does the swizzled
// layout: every thread rewrites 16-byte pieces where they lie.  The MMAs read the tile through the
// async proxy, hence the proxy fence before the tile is handed on.
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t w) {
  const float lo = __uint_as_float(w << 16), hi = __uint_as_float(w & 0xffff0000u);
  uint32_t r;
  asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
template <int kTile>
__device__ __forceinline__ void convert_tiles(const Work& w, const Args& a, uint32_t sbase, const Bars& bars, int cw,
                                              const Waiter& wt) {
  using T = TileGeo<kTile>;
  constexpr int kShare = T::kStage / kConvWarps;             // bytes per warp and tile
  constexpr int kPieces = kShare / (16 * 32);                // 16-byte pieces per lane
  static_assert(kShare % (16 * 32) == 0 && kPieces % 4 == 0, "tile does not split over the converting warps");
  const int lane = threadIdx.x & 31, S = a.n_stages;
  const uint32_t ring = sbase + (uint32_t)w.mb * 2u * 128u * 128u;
  Ring rs(S);
  for (int ti = 0; ti < w.nt; ++ti, rs.next()) {
    const int s = rs.i;
    if (!__all_sync(0xffffffffu, wt.wait(bars.k_full(s), rs.phase))) break;
    const uint32_t p0 = ring + s * T::kStage + cw * kShare + lane * 16;
#pragma unroll
    for (int it = 0; it < kPieces; it += 4) {
      uint4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) v[u] = lds128(p0 + (it + u) * 512);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        v[u].x = bf16x2_to_f16x2(v[u].x);
        v[u].y = bf16x2_to_f16x2(v[u].y);
        v[u].z = bf16x2_to_f16x2(v[u].z);
        v[u].w = bf16x2_to_f16x2(v[u].w);
        sts128(p0 + (it + u) * 512, v[u]);
      }
    }
    fence_proxy_async();
    __syncwarp();
    if (lane == 0) mbar_arrive(bars.k_conv(s));
  }
}

// The MMA issuer's last act when the CTA is aborting: see every MMA it issued retire before tensor
// memory is given back.
__device__ __forceinline__ void mma_drain(const Bars& bars) {
  tc_commit(bars.drain());
  drain_wait(bars.drain(), 0, kWaitLimit);
}

}  // namespace qg
}  // namespace dapq
