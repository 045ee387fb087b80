// Importance scoring on the 5th-generation tensor cores (Section 4.2, Eq. 4):
//   S(j) = sum_i Attention(q_i, k_j),  Attention = softmax(q K^T / sqrt(d_k)),
// summed over the G query heads of a GQA group, for bf16 caches.
//
// The G*N pseudo queries of one KV head form a dense [G*N x d] block that is scored
// against every key of that head: a contraction with G*N flop per byte of K, far above the
// HBM ridge, so the work belongs on tcgen05.mma with the accumulators in tensor memory.
// One exponential is owed per (query, key) pair and per sweep, which makes the MUFU/ALU
// pipes the co-limiter: the epilogue is kept to one FFMA + one ex2 + one FADD per pair.
//
// Two sweeps (column sums of a row-normalised matrix need every row's normaliser first):
//   sweep 1   D[query, key] = Q_blk K_tile^T   queries on TMEM lanes: each thread owns one
//             pseudo query and keeps its running max / sum of exp -> partials per chunk;
//   sweep 2   D[key, query] = K_tile Q_blk^T   keys on TMEM lanes: each thread owns one key
//             and sums exp2(s - lse_i) over the query columns -> scores, coalesced store.
//             Its epilogue threads first merge the partials of sweep 1 into the log-sum-exp
//             of the resident query rows (kept in shared memory), so no kernel runs between
//             the sweeps.
// The rotated queries are used as a bf16 pair (hi + lo, lo = bf16(q - hi)): two MMAs per
// k-step with the same K tile.  A single bf16 rounding of q would put the per-token scores
// of caches with outlier channels outside the 2e-3 tolerance.
//
// CTA = (chunk of 128-key tiles, KV head); 10 warps: warp 0 issues TMA loads (K tiles
// through a 3-stage ring, the query group once), warp 1 issues the MMAs and owns tensor
// memory, warps 2-9 are two epilogue groups (4 warps = 128 TMEM lanes each).  An accumulator
// job is a [128 x 128] fp32 block; four fit in tensor memory, so the MMA warp runs up to
// four jobs ahead of the epilogue, which reads each block in 32-column pieces with the next
// piece's load in flight while the current one is exponentiated.  Every mbarrier wait is
// bounded: after ~1 s the CTA raises the timeout status, drains and returns normally.
#include <cuda.h>
#include <math_constants.h>

#include "dapq_internal.cuh"

namespace dapq {
namespace {

constexpr int kTileKeys = 128;                 // keys per K tile (= UMMA M in sweep 2, N in sweep 1)
constexpr int kGroupRows = 256;                // query rows resident per group (2 M-blocks)
constexpr int kStages = 3;                     // K ring depth
constexpr int kHalfBytesK = kTileKeys * 128;   // one 64-channel half of a K tile (128-byte rows)
constexpr int kTileBytes = 2 * kHalfBytesK;    // 32 KB
constexpr int kHalfBytesQ = kGroupRows * 128;  // one half of a query group (32 KB)
constexpr int kQBytes = 2 * kHalfBytesQ;       // 64 KB per precision part (hi / lo)
constexpr int kThreads = 320;
constexpr int kTmemCols = 512;
constexpr long long kWaitLimit = 2000000000LL; // cycles (~1 s)

struct Smem {
  // offsets from the 1024-aligned base
  static constexpr int q_hi = 0;
  static constexpr int q_lo = q_hi + kQBytes;
  static constexpr int k = q_lo + kQBytes;
  static constexpr int bars = k + kStages * kTileBytes;
  // barriers: k_full[3], k_empty[3], acc_full[4], acc_empty[4], q_full, q_empty  (16 x 8 B)
  static constexpr int lse = bars + 16 * 8;          // [256] floats
  static constexpr int tmem_ptr = lse + kGroupRows * 4;
  static constexpr int abort_flag = tmem_ptr + 4;
  static constexpr int total = abort_flag + 4;
};
constexpr int kSmemBytes = Smem::total + 1024;   // slack for the manual 1024-byte alignment

// ------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the CTA is aborting (this or another wait ran out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  if (mbar_try(bar, parity)) return true;
  const long long start = clock64();
  while (true) {
    if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - start > kWaitLimit) {
      *abort_flag = 1;
      atomicOr(status, kStatusTimeout);
      return false;
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Shared-memory operand descriptor: K-major rows of 128 bytes, 128-byte swizzle, 8-row
// groups 1024 bytes apart (the layout a TMA box of 64 bf16 x rows with SWIZZLE_128B writes).
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3ffffu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, shape M x N.
__host__ __device__ constexpr uint32_t umma_idesc(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Three-input maximum (one instruction on sm_100).
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
// Wait for this thread's outstanding tensor-memory loads.  The registers of the load being
// waited for are passed through so that no use of them can be scheduled above the wait.
__device__ __forceinline__ void tmem_ld_wait_for(uint32_t* r) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                 "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
                 "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :: "memory");
}
// Barrier among the 8 epilogue warps only (the producer warps never join it).
__device__ __forceinline__ void epilogue_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

struct UmmaArgs {
  int32_t n_pseudo, group, n_q_heads, n_kv_heads;
  int32_t rows_total;        // G * N
  int32_t n_qgroups;         // ceil(rows_total / 256)
  int32_t has_lo;            // the query operand carries a low-order bf16 part
  int32_t lo_row_offset;     // rows between the hi and the lo copy in the query tensor
  float scale_log2e;
  float2* part;              // [n_chunks, H_kv, 2, n_qgroups * 256] (running max, sum) in base 2
  const float* lse_in;       // [B, H_q, N] natural-log lse from the caller, or NULL (use part)
  float* lse_out;            // [B, H_q, N] natural-log lse used, or NULL
  float* scores;
  int64_t score_stride;
  int* status;
};

// One accumulator job is a [128 x 128] fp32 block in tensor memory (4 of them fit):
//   sweep 1: 128 pseudo queries (lanes) x 128 keys (columns);
//   sweep 2: 128 keys (lanes) x 128 pseudo queries (columns).
constexpr int kAccBufs = 4;
constexpr int kAccCols = kTmemCols / kAccBufs;

template <bool kSweep2>
__global__ void __launch_bounds__(kThreads, 1)
score_umma_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_q,
                  const __grid_constant__ SeqTable t, const __grid_constant__ ChunkTable ct, const UmmaArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- this CTA's work: KV head, sequence, tile range
  const int chunk = blockIdx.x, kvh = blockIdx.y;
  const int b = find_segment(ct.cu_chunk, t.batch, chunk);
  const int L = t.prompt_len[b], N = a.n_pseudo;
  const int n_tiles = (L + N + kTileKeys - 1) / kTileKeys;
  const int t0 = (chunk - ct.cu_chunk[b]) * ct.chunk_tiles;
  int t1 = min(n_tiles, t0 + ct.chunk_tiles);
  if (kSweep2) t1 = min(t1, (L + kTileKeys - 1) / kTileKeys);   // tiles of synthetic keys give no score
  const int nt = t1 - t0;
  if (nt <= 0) return;
  const int row_base = t.cu_rows[b];                            // first cache row of the sequence
  const int qrow_base = (b * a.n_q_heads + kvh * a.group) * N;  // first query row of this KV head

  const uint32_t bar0 = sbase + Smem::bars;
  auto k_full = [&](int s) { return bar0 + 8u * s; };
  auto k_empty = [&](int s) { return bar0 + 8u * (3 + s); };
  auto acc_full = [&](int i) { return bar0 + 8u * (6 + i); };
  auto acc_empty = [&](int i) { return bar0 + 8u * (10 + i); };
  const uint32_t q_full = bar0 + 8u * 14, q_empty = bar0 + 8u * 15;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + Smem::abort_flag);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + Smem::tmem_ptr);
  float* lse_s = reinterpret_cast<float*>(smem + Smem::lse);    // [256] base-2 lse of the resident query group

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(k_full(s), 1); mbar_init(k_empty(s), 1); }
    for (int i = 0; i < 4; ++i) { mbar_init(acc_full(i), 1); mbar_init(acc_empty(i), 4); }
    mbar_init(q_full, 1);
    mbar_init(q_empty, 1);
    *abort_flag = 0;
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
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // =========================================================================== TMA producer
    if (lane == 0) {
      int li = 0;                                               // K tiles loaded so far
      bool ok = true;
      for (int qg = 0; qg < a.n_qgroups && ok; ++qg) {
        const int rows_g = min(kGroupRows, a.rows_total - qg * kGroupRows);
        const int mb = (rows_g + 127) / 128;
        if (qg > 0) ok = mbar_wait(q_empty, (qg - 1) & 1, abort_flag, a.status);
        if (!ok) break;
        const int parts = a.has_lo ? 2 : 1;
        mbar_expect_tx(q_full, (uint32_t)(parts * mb * 2 * 128 * 128));
        for (int part = 0; part < parts; ++part)
          for (int half = 0; half < 2; ++half)
            for (int m = 0; m < mb; ++m)
              tma_load_2d(sbase + (part ? Smem::q_lo : Smem::q_hi) + half * kHalfBytesQ + m * 128 * 128, &tm_q, q_full,
                          half * 64, part * a.lo_row_offset + qrow_base + qg * kGroupRows + m * 128);
        for (int ti = 0; ti < nt; ++ti, ++li) {
          const int s = li % kStages;
          if (li >= kStages) ok = mbar_wait(k_empty(s), ((li / kStages) - 1) & 1, abort_flag, a.status);
          if (!ok) break;
          mbar_expect_tx(k_full(s), kTileBytes);
          const int row = row_base + (t0 + ti) * kTileKeys;
          tma_load_3d(sbase + Smem::k + s * kTileBytes, &tm_k, k_full(s), 0, row, kvh);
          tma_load_3d(sbase + Smem::k + s * kTileBytes + kHalfBytesK, &tm_k, k_full(s), 64, row, kvh);
        }
      }
      if (!ok) {
        // aborting: let the copies already issued land before the CTA returns
        for (int back = 1; back <= kStages && back <= li; ++back) {
          const int l2 = li - back;
          const long long start = clock64();
          while (!mbar_try(k_full(l2 % kStages), (l2 / kStages) & 1) && clock64() - start < kWaitLimit) {}
        }
      }
    }
  } else if (warp == 1) {
    // ============================================================================= MMA issuer
    if (lane == 0) {
      int li = 0, job = 0;
      bool ok = true;
      for (int qg = 0; qg < a.n_qgroups && ok; ++qg) {
        const int rows_g = min(kGroupRows, a.rows_total - qg * kGroupRows);
        const int mb = (rows_g + 127) / 128;
        ok = mbar_wait(q_full, qg & 1, abort_flag, a.status);
        for (int ti = 0; ti < nt && ok; ++ti, ++li) {
          const int s = li % kStages;
          ok = mbar_wait(k_full(s), (li / kStages) & 1, abort_flag, a.status);
          if (!ok) break;
          const uint32_t kaddr = sbase + Smem::k + s * kTileBytes;
          for (int m = 0; m < mb && ok; ++m, ++job) {
            const int buf = job % kAccBufs;
            if (job >= kAccBufs) ok = mbar_wait(acc_empty(buf), ((job / kAccBufs) - 1) & 1, abort_flag, a.status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d = tmem_base + buf * kAccCols;
            // sweep 2: only the query columns that exist (rounded up to the MMA's N granule of 16)
            const int n2 = (min(128, rows_g - m * 128) + 15) & ~15;
            const uint32_t idesc = kSweep2 ? umma_idesc(128, n2) : umma_idesc(128, kTileKeys);
            uint32_t accum = 0;
            for (int part = 0; part < (a.has_lo ? 2 : 1); ++part) {
              const uint32_t qaddr = sbase + (part ? Smem::q_lo : Smem::q_hi) + m * 128 * 128;
#pragma unroll
              for (int ks = 0; ks < 8; ++ks) {
                const int half = ks >> 2, kk = ks & 3;
                const uint64_t kd = umma_desc(kaddr + half * kHalfBytesK + kk * 32);
                const uint64_t qd = umma_desc(qaddr + half * kHalfBytesQ + kk * 32);
                if (kSweep2) umma(d, kd, qd, idesc, accum); else umma(d, qd, kd, idesc, accum);
                accum = 1;
              }
            }
            tc_commit(acc_full(buf));
          }
          tc_commit(k_empty(s));                                // the K stage is free once these MMAs retire
        }
        tc_commit(q_empty);
      }
    }
  } else {
    // ============================================================================== epilogue
    const int eg = (warp - 2) >> 2;                             // epilogue group 0 / 1
    const int quad = warp & 3;                                  // TMEM lane quadrant of this warp
    const int r = quad * 32 + lane;                             // accumulator row of this thread
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float c = a.scale_log2e;
    int job = 0;
    bool ok = true;
    // (an aborting group still walks every query group: the other group waits for it at the barriers)
    for (int qg = 0; qg < a.n_qgroups && (ok || kSweep2); ++qg) {
      const int rows_g = min(kGroupRows, a.rows_total - qg * kGroupRows);
      const int mb = (rows_g + 127) / 128;
      if (kSweep2) {
        // ---- base-2 log-sum-exp of the group's rows: thread (eg, r) merges the per-chunk
        // partials of row eg*128 + r in a fixed order, or converts the caller's value
        if (qg > 0) epilogue_sync();                            // the previous group's values are no longer read
        {
          const int row = eg * 128 + r, grow = qg * kGroupRows + row;
          float l2 = 0.f;
          if (grow < a.rows_total) {
            if (a.lse_in) {
              l2 = a.lse_in[qrow_base + grow] * 1.4426950408889634f;
            } else {
              const int rows_pad = a.n_qgroups * kGroupRows;
              const float2* p = a.part + ((int64_t)ct.cu_chunk[b] * a.n_kv_heads + kvh) * 2 * rows_pad + grow;
              const int64_t step = (int64_t)a.n_kv_heads * 2 * rows_pad;
              const int nc = ct.cu_chunk[b + 1] - ct.cu_chunk[b];
              float mx = -CUDART_INF_F;
              for (int cc = 0; cc < nc; ++cc) {
                mx = fmaxf(mx, p[cc * step].x);
                mx = fmaxf(mx, p[cc * step + rows_pad].x);
              }
              float z = 0.f;
              for (int cc = 0; cc < nc; ++cc) {
                const float2 p0 = p[cc * step], p1 = p[cc * step + rows_pad];
                z += p0.y * exp2f(p0.x - mx);
                z += p1.y * exp2f(p1.x - mx);
              }
              l2 = mx + log2f(z);
            }
            if (a.lse_out && chunk == ct.cu_chunk[b]) a.lse_out[qrow_base + grow] = l2 * 0.6931471805599453f;
          }
          lse_s[row] = l2;
        }
        epilogue_sync();
        // Tile ti always goes to group ti & 1, so one thread owns a key's score across both
        // column blocks and all query groups and accumulates it in program order.
        for (int ti = 0; ti < nt && ok; ++ti) {
          if ((ti & 1) != eg) { job += mb; continue; }
          float sum0 = 0.f, sum1 = 0.f;
          for (int m = 0; m < mb && ok; ++m, ++job) {
            const int buf = job % kAccBufs;
            ok = __all_sync(0xffffffffu, mbar_wait(acc_full(buf), (job / kAccBufs) & 1, abort_flag, a.status));
            if (!ok) break;
            tc_fence_after();
            const int cols = min(128, rows_g - m * 128);        // query columns of this block
            const int nch = (cols + 31) >> 5;
            const uint32_t taddr = lane_addr + buf * kAccCols;
            const float* lse_m = lse_s + m * 128;
            uint32_t v[2][32];
            tmem_ld32(taddr, v[0]);
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
              if (ch < nch) {
                tmem_ld_wait_for(v[ch & 1]);
                if (ch + 1 < nch) tmem_ld32(taddr + (ch + 1) * 32, v[(ch + 1) & 1]);
                const int valid = cols - ch * 32;               // >= 32 except in the last chunk
                if (valid >= 32) {
#pragma unroll
                  for (int e = 0; e < 32; e += 4) {
                    const float4 l4 = *reinterpret_cast<const float4*>(lse_m + ch * 32 + e);
                    sum0 += ex2(fmaf(__uint_as_float(v[ch & 1][e]), c, -l4.x));
                    sum1 += ex2(fmaf(__uint_as_float(v[ch & 1][e + 1]), c, -l4.y));
                    sum0 += ex2(fmaf(__uint_as_float(v[ch & 1][e + 2]), c, -l4.z));
                    sum1 += ex2(fmaf(__uint_as_float(v[ch & 1][e + 3]), c, -l4.w));
                  }
                } else {
#pragma unroll
                  for (int e = 0; e < 32; ++e)
                    if (e < valid) sum0 += ex2(fmaf(__uint_as_float(v[ch & 1][e]), c, -lse_m[ch * 32 + e]));
                }
              }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty(buf));
          }
          if (!ok) break;
          const int j = (t0 + ti) * kTileKeys + r;              // sequence-local key position
          if (j < L) {
            float* out = a.scores + (int64_t)kvh * a.score_stride + t.cu_prompt[b] + j;
            const float sum = sum0 + sum1;
            *out = (qg == 0) ? sum : *out + sum;
          }
        }
      } else {
        float m_raw = -CUDART_INF_F, z = 0.f;                   // running max (raw dot product) and sum
        const int i_row = (qg * kGroupRows + r) % N;            // pseudo-query index if this thread's block is 0
        for (int ti = 0; ti < nt && ok; ++ti) {
          const int tile_base = (t0 + ti) * kTileKeys;
          const bool masked = tile_base + kTileKeys > L;        // holds synthetic (or foreign) rows
          for (int m = 0; m < mb && ok; ++m, ++job) {
            if ((job & 1) != eg) continue;
            const int buf = job % kAccBufs;
            ok = __all_sync(0xffffffffu, mbar_wait(acc_full(buf), (job / kAccBufs) & 1, abort_flag, a.status));
            if (!ok) break;
            tc_fence_after();
            // key column `col` of this tile is visible to pseudo query i iff its position <= L + i
            const int i = (i_row + m * 128) % N;
            const int lim = L + i - tile_base;                  // last visible column
            const uint32_t taddr = lane_addr + buf * kAccCols;
            uint32_t v[2][32];
            tmem_ld32(taddr, v[0]);
#pragma unroll
            for (int ch = 0; ch < kTileKeys / 32; ++ch) {
              tmem_ld_wait_for(v[ch & 1]);
              if (ch + 1 < kTileKeys / 32) tmem_ld32(taddr + (ch + 1) * 32, v[(ch + 1) & 1]);
              float x[32];
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                x[e] = __uint_as_float(v[ch & 1][e]);
                if (masked && ch * 32 + e > lim) x[e] = -CUDART_INF_F;
              }
              float cmax = max3(x[0], x[1], x[2]);
#pragma unroll
              for (int e = 3; e < 31; e += 2) cmax = max3(cmax, x[e], x[e + 1]);
              cmax = fmaxf(cmax, x[31]);
              if (cmax > m_raw) {
                z *= ex2((m_raw - cmax) * c);
                m_raw = cmax;
              }
              if (m_raw > -CUDART_INF_F) {
                const float neg = -m_raw * c;
                float s0 = 0.f, s1 = 0.f;
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                  s0 += ex2(fmaf(x[e], c, neg));
                  s1 += ex2(fmaf(x[e + 1], c, neg));
                }
                z += s0 + s1;
              }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty(buf));
          }
        }
        // partials: slot eg of every row this group may own; neutral where it had no job
        float2* pbase = a.part + (((int64_t)chunk * a.n_kv_heads + kvh) * 2 + eg) * (a.n_qgroups * kGroupRows) +
                        qg * kGroupRows;
        for (int m = 0; m < mb; ++m) {
          const bool mine = (mb == 1) || (m == eg);             // with 2 blocks, group e takes block e
          if (qg * kGroupRows + m * 128 + r < a.rows_total)
            pbase[m * 128 + r] = mine ? make_float2(m_raw * c, z) : make_float2(-CUDART_INF_F, 0.f);
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

bool encode_bf16_map(CUtensorMap* map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t gdim[3], gstride[2];
  cuuint32_t box[3] = {64, (cuuint32_t)kTileKeys, 1}, estr[3] = {1, 1, 1};
  for (int i = 0; i < rank; ++i) gdim[i] = dims[i];
  for (int i = 0; i < rank - 1; ++i) gstride[i] = strides_bytes[i];
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool plan_umma_chunks(const SeqTable& t, int n_pseudo, int n_kv_heads, int n_sm, ChunkTable* ct) {
  int64_t total_tiles = 0;
  int max_tiles = 0;
  for (int b = 0; b < t.batch; ++b) {
    const int tiles = (t.prompt_len[b] + n_pseudo + kTileKeys - 1) / kTileKeys;
    total_tiles += tiles;
    max_tiles = tiles > max_tiles ? tiles : max_tiles;
  }
  // cost of a candidate = waves of CTAs x (tiles per CTA + fixed per-CTA work, in tile units)
  int best_c = 0;
  double best_cost = 0.0;
  for (int c = 1; c <= max_tiles; ++c) {
    int64_t n = 0;
    for (int b = 0; b < t.batch; ++b) {
      const int tiles = (t.prompt_len[b] + n_pseudo + kTileKeys - 1) / kTileKeys;
      n += (tiles + c - 1) / c;
    }
    if (n > t.batch + kUmmaMaxChunks) continue;
    const int64_t waves = (n * n_kv_heads + n_sm - 1) / n_sm;
    const double cost = (double)waves * (c + 3.0);
    if (best_c == 0 || cost < best_cost) { best_c = c; best_cost = cost; }
  }
  if (best_c == 0) return false;
  ct->chunk_tiles = best_c;
  int32_t n = 0;
  for (int b = 0; b < t.batch; ++b) {
    const int tiles = (t.prompt_len[b] + n_pseudo + kTileKeys - 1) / kTileKeys;
    ct->cu_chunk[b] = n;
    n += (tiles + best_c - 1) / best_c;
  }
  ct->cu_chunk[t.batch] = n;
  ct->n_chunks = n;
  return true;
}

}  // namespace

int64_t umma_part_elems(int max_batch, int n_q_heads, int n_kv_heads, int n_pseudo) {
  const int rows_total = n_q_heads / n_kv_heads * n_pseudo;
  const int rows_pad = (rows_total + kGroupRows - 1) / kGroupRows * kGroupRows;
  return (int64_t)(max_batch + kUmmaMaxChunks) * n_kv_heads * 2 * rows_pad;
}

bool umma_plan(const void* q_hi, int has_lo, int64_t lo_row_offset, const CacheDev& cv, const SeqTable& t,
               const Dims& dm, int n_sm, UmmaPlan* plan) {
  if (!plan_umma_chunks(t, dm.n_pseudo, dm.n_kv_heads, n_sm, &plan->ct)) return false;
  plan->has_lo = has_lo;
  plan->lo_row_offset = lo_row_offset;
  // ---- tensor maps: K as [d, rows, H_kv], the query operand as [d, rows]
  const uint64_t rows_k = (uint64_t)t.cu_rows[t.batch];
  const uint64_t kd[3] = {(uint64_t)kHeadDim, rows_k, (uint64_t)dm.n_kv_heads};
  uint64_t ks[2] = {(uint64_t)cv.k_row_stride * 2, (uint64_t)cv.k_head_stride * 2};
  if (dm.n_kv_heads == 1 && ks[1] == 0) ks[1] = ks[0] * rows_k;
  const uint64_t q_rows = (uint64_t)t.batch * dm.n_q_heads * dm.n_pseudo;
  const uint64_t qd[2] = {(uint64_t)kHeadDim, has_lo ? (uint64_t)lo_row_offset + q_rows : q_rows};
  const uint64_t qs[1] = {(uint64_t)kHeadDim * 2};
  if (ks[1] == 0 || ks[1] % 16) return false;
  return encode_bf16_map(&plan->tm_k, cv.k, 3, kd, ks) && encode_bf16_map(&plan->tm_q, q_hi, 2, qd, qs);
}

cudaError_t launch_score_umma(const UmmaPlan& plan, const SeqTable& t, const Dims& dm, const float* lse_in,
                              float2* part, float* scores, int64_t score_stride, float* lse_out,
                              int* status, cudaStream_t s, LaunchLog* log) {
  const ChunkTable& ct = plan.ct;
  UmmaArgs a;
  a.n_pseudo = dm.n_pseudo;
  a.group = dm.group;
  a.n_q_heads = dm.n_q_heads;
  a.n_kv_heads = dm.n_kv_heads;
  a.rows_total = dm.group * dm.n_pseudo;
  a.n_qgroups = (a.rows_total + kGroupRows - 1) / kGroupRows;
  a.has_lo = plan.has_lo;
  a.lo_row_offset = (int32_t)plan.lo_row_offset;
  a.scale_log2e = dm.scale_log2e;
  a.part = part;
  a.lse_in = lse_in;
  a.lse_out = lse_out;
  a.scores = scores;
  a.score_stride = score_stride;
  a.status = status;

  auto k1 = score_umma_kernel<false>;
  auto k2 = score_umma_kernel<true>;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes)) != cudaSuccess) return e;
  const dim3 grid(ct.n_chunks, dm.n_kv_heads);
  if (lse_in == nullptr) {
    log->begin(kKindSweep1, s);
    k1<<<grid, kThreads, kSmemBytes, s>>>(plan.tm_k, plan.tm_q, t, ct, a);
    log->end(s);
  }
  log->begin(kKindSweep2, s);
  k2<<<grid, kThreads, kSmemBytes, s>>>(plan.tm_k, plan.tm_q, t, ct, a);
  log->end(s);
  return cudaGetLastError();
}

}  // namespace dapq
