// Definitions shared by the two sweeps of the tensor-core scorer (see score_umma.cu).
#pragma once
#include "umma_ptx.cuh"

namespace dapq {
namespace umma {

using namespace ptx;

constexpr int kTile1 = 192;                    // keys per K tile of sweep 1 (= UMMA N there)
constexpr int kTile2 = 128;                    // keys per K tile of sweep 2 (= UMMA M there)
constexpr int kEpiGroups = 4;                  // epilogue groups of 4 warps (128 TMEM lanes each)
constexpr int kThreads = 64 + kEpiGroups * 128;
constexpr int kTmemCols = 512;
constexpr int kStageBytes1 = kTile1 * 256, kHalfBytes1 = kTile1 * 128;   // one K tile of sweep 1 / its 64-channel half
constexpr int kStageBytes2 = kTile2 * 256, kHalfBytes2 = kTile2 * 128;

// Geometry of a CTA.  kCompact = the G*N query rows of a KV head fit one block of 128 (the
// paper's default window, N = 32 with four query heads per KV head): the query operand then
// takes 64 KB instead of 128 KB, sweep 1 (which streams K from DRAM) gets a third K stage, and
// sweep 2 runs four accumulators of 128 columns instead of two of 256.
template <bool kCompact>
struct Geo {
  static constexpr int kRows = kCompact ? 128 : 256;          // query rows resident per group
  static constexpr int kHalfBytesQ = kRows * 128;             // one 64-channel half of a query group
  static constexpr int kQBytes = 2 * kHalfBytesQ;             // per precision part (hi / lo)
  static constexpr int kRingBytes = 224 * 1024 - 2 * kQBytes;
  static constexpr int kStages1 = kRingBytes / kStageBytes1;  // 2 / 3 tiles of 192 keys
  static constexpr int kStages2 = 3;                          // tiles of 128 keys (a deeper ring slows sweep 2 down:
                                                              // its MMAs already take most of the shared-memory bandwidth)
  static constexpr int kAcc2 = kCompact ? 4 : 2;              // accumulators of sweep 2
  static constexpr int kAccCols2 = kTmemCols / kAcc2;
  // shared memory (offsets from the 1024-aligned base): query group as a bf16 pair, K ring
  static constexpr int q_hi = 0;
  static constexpr int q_lo = kQBytes;
  static constexpr int k = 2 * kQBytes;
};
constexpr int kMaxStages = 3, kMaxAcc = 4;
// ... followed, at the same place in both geometries, by the barriers, the group's log-sum-exp
// (sweep 2) and two words.
struct Smem {
  static constexpr int bars = 224 * 1024;
  // barriers (18 x 8 B): k_full[3], k_empty[3], acc_full[4], acc_empty[4], q_full, q_empty, part_full, part_empty
  static constexpr int lse = bars + 18 * 8;          // [256] floats
  static constexpr int exch = lse + 256 * 4;         // [3][128] floats: the partial sums of epilogue groups 1-3 (sweep 2);
                                                     // lse + exch together: [256] float2 row statistics (sweep 1)
  static constexpr int tmem_ptr = exch + 3 * 128 * 4;
  static constexpr int abort_flag = tmem_ptr + 4;
  static constexpr int total = abort_flag + 4;
};
static_assert(Geo<false>::k + Geo<false>::kStages1 * kStageBytes1 <= Smem::bars && Geo<true>::k + Geo<true>::kStages1 * kStageBytes1 <= Smem::bars &&
              Geo<false>::k + Geo<false>::kStages2 * kStageBytes2 <= Smem::bars && Geo<true>::k + Geo<true>::kStages2 * kStageBytes2 <= Smem::bars,
              "K ring overruns the barriers");
static_assert(Geo<true>::kStages1 <= kMaxStages && Geo<true>::kStages2 <= kMaxStages && Geo<true>::kAcc2 <= kMaxAcc, "barrier table too small");
// The kernels declare their dynamic shared memory 1024-byte aligned (what the 128-byte swizzle of the
// TMA / UMMA tiles needs) and check it: a CTA that finds it otherwise raises a status bit and returns.
constexpr int kSmemBytes = Smem::total;
static_assert(kSmemBytes <= 232448, "exceeds the shared memory a CTA can opt in to");

struct UmmaArgs {
  int32_t n_pseudo, group, n_q_heads, n_kv_heads;
  int32_t rows_total;        // G * N
  int32_t n_qgroups;         // ceil(rows_total / rows per group)
  int32_t rows_pad;          // n_qgroups * rows per group
  int32_t has_lo;            // the query operand carries a low-order bf16 part
  int32_t lo_row_offset;     // rows between the hi and the lo copy in the query tensor
  float scale_log2e;
  long long wait_limit;      // cycles a wait may take before the CTA gives up
  float2* part;              // [n_chunks1, H_kv, rows_pad] (running max, sum) of every query row over a chunk's keys, base 2
  const float* lse_in;       // [B, H_q, N] natural-log lse from the caller, or NULL (use part)
  float* lse_out;            // [B, H_q, N] natural-log lse used, or NULL
  float* scores;
  int64_t score_stride;
  int* status;
};

// This CTA's work: sequence, tile range, first cache row and first query row.
struct Work {
  int b, L, nt, t0, row_base, qrow_base;
};
// n_keys(b): keys of sequence b that the sweep covers (L_b + N in sweep 1, L_b in sweep 2).
__device__ __forceinline__ Work cta_work(const SeqTable& t, const ChunkTable& ct, const UmmaArgs& a, int tile_keys,
                                         bool with_synthetic) {
  Work w;
  const int chunk = blockIdx.x, kvh = blockIdx.y;
  w.b = find_segment(ct.cu_chunk, t.batch, chunk);
  w.L = t.prompt_len[w.b];
  const int n_keys = w.L + (with_synthetic ? a.n_pseudo : 0);
  const int n_tiles = (n_keys + tile_keys - 1) / tile_keys;
  w.t0 = (chunk - ct.cu_chunk[w.b]) * ct.chunk_tiles;
  w.nt = min(n_tiles, w.t0 + ct.chunk_tiles) - w.t0;
  w.row_base = t.cu_rows[w.b];                                          // first cache row of the sequence
  w.qrow_base = (w.b * a.n_q_heads + kvh * a.group) * a.n_pseudo;       // first query row of this KV head
  return w;
}

// Barrier addresses of a CTA.
struct Bars {
  uint32_t base;
  __device__ __forceinline__ uint32_t k_full(int s) const { return base + 8u * s; }
  __device__ __forceinline__ uint32_t k_empty(int s) const { return base + 8u * (kMaxStages + s); }
  __device__ __forceinline__ uint32_t acc_full(int i) const { return base + 8u * (2 * kMaxStages + i); }
  __device__ __forceinline__ uint32_t acc_empty(int i) const { return base + 8u * (2 * kMaxStages + kMaxAcc + i); }
  __device__ __forceinline__ uint32_t q_full() const { return base + 8u * (2 * kMaxStages + 2 * kMaxAcc); }
  __device__ __forceinline__ uint32_t q_empty() const { return base + 8u * (2 * kMaxStages + 2 * kMaxAcc + 1); }
  __device__ __forceinline__ uint32_t part_full() const { return base + 8u * (2 * kMaxStages + 2 * kMaxAcc + 2); }
  __device__ __forceinline__ uint32_t part_empty() const { return base + 8u * (2 * kMaxStages + 2 * kMaxAcc + 3); }
};

// Common CTA prologue: barrier init, tensor-memory allocation (warp 1), one CTA-wide sync, then
// the wait for the kernel before this one (its set-up overlaps that kernel's tail).
// Returns the tensor-memory base address.
__device__ __forceinline__ uint32_t cta_prologue(uint8_t* smem, uint32_t sbase, const Bars& bars, int n_stages, int n_acc) {
  const int warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stages; ++s) { mbar_init(bars.k_full(s), 1); mbar_init(bars.k_empty(s), 1); }
    for (int i = 0; i < n_acc; ++i) {
      mbar_init(bars.acc_full(i), 1);
      mbar_init(bars.acc_empty(i), 4 * kEpiGroups);        // every epilogue warp reads every accumulator
    }
    mbar_init(bars.part_full(), 4 * (kEpiGroups - 1));     // the groups that hand their partial sums to group 0
    mbar_init(bars.part_empty(), 4);                       // group 0 has read them
    mbar_init(bars.q_full(), 1);
    mbar_init(bars.q_empty(), 1);
    *reinterpret_cast<volatile int*>(smem + Smem::abort_flag) = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {                                              // tensor memory: all 512 columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(sbase + Smem::tmem_ptr), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();                                                   // global memory is touched only from here on
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

// TMA producer loop shared by both sweeps: per query group the query blocks (hi, lo), then the
// CTA's K tiles through the ring.  kTile / kStages / kHalf are the sweep's tile geometry.
// kSideBySide (compact geometry only): per 64-channel half, the 128 hi rows are followed directly by the
// 128 lo rows, so that one MMA of N = 256 reads both.
template <class G, int kTile, int kStages, int kStage, int kHalf, bool kSideBySide = false>
__device__ __forceinline__ void tma_producer(const CUtensorMap* tm_k, const CUtensorMap* tm_q, const Work& w,
                                             const UmmaArgs& a, uint32_t sbase, const Bars& bars, int kvh,
                                             volatile int* abort_flag) {
  int li = 0, n_q = 0;                                      // K tiles / query groups loaded so far
  bool ok = true;
  auto load_tile = [&](int ti) {
    const int s = li % kStages;
    mbar_expect_tx(bars.k_full(s), kStage);
    const int row = w.row_base + (w.t0 + ti) * kTile;
    tma_load_3d(sbase + G::k + s * kStage, tm_k, bars.k_full(s), 0, row, kvh);
    tma_load_3d(sbase + G::k + s * kStage + kHalf, tm_k, bars.k_full(s), 64, row, kvh);
    ++li;
  };
  // The first K tile goes out before the queries (it comes from further away: DRAM in sweep 1); the
  // rest of the ring follows them, so that the first job's operands are not queued behind tiles that
  // later jobs need (measured: sweep 2 starts 1 us earlier than with the whole ring ahead of the queries).
  const int n_first = min(1, w.nt);
  for (int ti = 0; ti < n_first; ++ti) load_tile(ti);
  for (int qg = 0; qg < a.n_qgroups && ok; ++qg) {
    const int rows_g = min(G::kRows, a.rows_total - qg * G::kRows);
    const int mb = (rows_g + 127) / 128;
    if (qg > 0) ok = mbar_wait_limit(bars.q_empty(), (qg - 1) & 1, abort_flag, a.status, a.wait_limit);
    if (!ok) break;
    const int parts = a.has_lo ? 2 : 1;
    mbar_expect_tx(bars.q_full(), (uint32_t)(parts * mb * 2 * 128 * 128));
    ++n_q;
    for (int part = 0; part < parts; ++part)
      for (int half = 0; half < 2; ++half)
        for (int m = 0; m < mb; ++m)
          tma_load_2d(sbase + (kSideBySide ? half * 2 * G::kHalfBytesQ + part * G::kHalfBytesQ
                                           : (part ? G::q_lo : G::q_hi) + half * G::kHalfBytesQ + m * 128 * 128),
                      tm_q, bars.q_full(), half * 64, part * a.lo_row_offset + w.qrow_base + qg * G::kRows + m * 128);
    for (int ti = (qg == 0 ? n_first : 0); ti < w.nt; ++ti) {
      const int s = li % kStages;
      if (li >= kStages) ok = mbar_wait_limit(bars.k_empty(s), ((li / kStages) - 1) & 1, abort_flag, a.status, a.wait_limit);
      if (!ok) break;
      load_tile(ti);
    }
  }
  // See every copy issued above land before this thread (and with it the CTA) returns: in a normal run they
  // have all been consumed by now; in an aborting CTA nobody else may be left to wait for them.
  for (int back = 1; back <= kStages && back <= li; ++back) {
    const int l2 = li - back;
    drain_wait(bars.k_full(l2 % kStages), (l2 / kStages) & 1, kWaitLimit);
  }
  if (n_q > 0) drain_wait(bars.q_full(), (n_q - 1) & 1, kWaitLimit);
}

// The MMA issuer's last act: see every MMA it issued retire before tensor memory is given back.  q_empty
// receives one commit per finished query group (n_done so far); an issuer that left its loop early adds one.
__device__ __forceinline__ void mma_drain(const Bars& bars, int n_done, bool left_early) {
  if (left_early) {
    tc_commit(bars.q_empty());
    ++n_done;
  }
  if (n_done > 0) drain_wait(bars.q_empty(), (n_done - 1) & 1, kWaitLimit);
}

}  // namespace umma
}  // namespace dapq
