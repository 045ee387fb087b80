// Importance scoring on the 5th-generation tensor cores (Section 4.2, Eq. 4):
//   S(j) = sum_i Attention(q_i, k_j),  Attention = softmax(q K^T / sqrt(d_k)),
// summed over the G query heads of a GQA group, for bf16 caches.
//
// The G*N pseudo queries of one KV head form a dense [G*N x d] block that is scored
// against every key of that head: a contraction with G*N flop per byte of K, far above the
// HBM ridge, so the work belongs on tcgen05.mma with the accumulators in tensor memory.
// One exponential is owed per (query, key) pair and per sweep, which makes the MUFU/ALU
// pipes the co-limiter: the epilogues are kept to a handful of instructions per pair.
//
// Two sweeps (column sums of a row-normalised matrix need every row's normaliser first):
//   sweep 1   D[query, key] = Q_blk K_tile^T   queries on TMEM lanes: each thread owns one
//             pseudo query and keeps its running max / sum of exp -> partials per chunk.
//             The query block is the A operand and lives in TENSOR MEMORY (written once per
//             CTA with tcgen05.st), so an MMA reads only the K slab from shared memory:
//             with both operands in shared memory the operand fetch saturates the
//             shared-memory bandwidth and the TMA writes of the next tiles starve.
//   sweep 2   D[key, query] = K_tile Q_grp^T   keys on TMEM lanes: each thread owns one key
//             and sums exp2(s - lse_i) over up to 256 query columns -> scores, coalesced
//             store.  N = 256 per MMA keeps the operand traffic at 3/4 of the bandwidth.
//             Its epilogue threads first merge the partials of sweep 1 into the log-sum-exp
//             of the resident query rows (kept in shared memory), so no kernel runs between
//             the sweeps.
// The rotated queries are used as a bf16 pair (hi + lo, lo = bf16(q - hi)): two MMAs per
// k-step with the same K tile.  A single bf16 rounding of q would put the per-token scores
// of caches with outlier channels outside the 2e-3 tolerance.
//
// CTA = (chunk of 128-key tiles, KV head); 10 warps: warp 0 issues the TMA loads of the K
// ring, warp 1 issues the MMAs and owns tensor memory, warps 2-9 are two epilogue groups
// (4 warps = 128 TMEM lanes each) that take alternate accumulators and read them in
// 32-column pieces with the next piece's load in flight while the current one is
// exponentiated.  Every mbarrier wait is bounded: after ~1 s the CTA raises the timeout
// status, drains and returns normally.
#include <cuda.h>
#include <math_constants.h>

#include "dapq_internal.cuh"

namespace dapq {
namespace {

constexpr int kTileKeys = 128;                 // keys per K tile (= UMMA M in sweep 2, N in sweep 1)
constexpr int kGroupRows = 256;                // query rows resident per group (2 blocks of 128)
constexpr int kHalfBytesK = kTileKeys * 128;   // one 64-channel half of a K tile (128-byte rows)
constexpr int kTileBytes = 2 * kHalfBytesK;    // 32 KB
constexpr int kHalfBytesQ = kGroupRows * 128;  // one half of a query group (32 KB)
constexpr int kQBytes = 2 * kHalfBytesQ;       // 64 KB per precision part (hi / lo)
constexpr int kThreads = 320;
constexpr int kTmemCols = 512;
constexpr long long kWaitLimit = 2000000000LL; // cycles (~1 s)

// Shared memory of sweep 1 (offsets from the 1024-aligned base): only the K ring.
constexpr int kStages1 = 6;
struct Smem1 {
  static constexpr int k = 0;
  static constexpr int bars = k + kStages1 * kTileBytes;
  // barriers: k_full[6], k_empty[6], acc_full[2], acc_empty[2], a_full  (17 x 8 B)
  static constexpr int tmem_ptr = bars + 17 * 8;
  static constexpr int abort_flag = tmem_ptr + 4;
  static constexpr int total = abort_flag + 4;
};
// Shared memory of sweep 2: the query group (hi and lo), a 3-stage K ring, the group's lse.
constexpr int kStages2 = 3;
struct Smem2 {
  static constexpr int q_hi = 0;
  static constexpr int q_lo = q_hi + kQBytes;
  static constexpr int k = q_lo + kQBytes;
  static constexpr int bars = k + kStages2 * kTileBytes;
  // barriers: k_full[3], k_empty[3], acc_full[2], acc_empty[2], q_full, q_empty  (12 x 8 B)
  static constexpr int lse = bars + 12 * 8;          // [256] floats
  static constexpr int tmem_ptr = lse + kGroupRows * 4;
  static constexpr int abort_flag = tmem_ptr + 4;
  static constexpr int total = abort_flag + 4;
};
constexpr int kSmemBytes1 = Smem1::total + 1024;   // slack for the manual 1024-byte alignment
constexpr int kSmemBytes2 = Smem2::total + 1024;

// Tensor-memory columns of sweep 1: the A operand (block m, part p at (2m + p) * 64) and
// one [128 x 128] accumulator per epilogue group.
constexpr int kACols = 64;                     // 128 bf16 channels = 64 32-bit columns
constexpr int kAcc1 = 256;                     // first accumulator column of sweep 1

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
// D (tensor memory) (+)= A (shared memory) B (shared memory)
__device__ __forceinline__ void umma_ss(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
}
// D (tensor memory) (+)= A (tensor memory: one row per lane, two bf16 per column) B (shared memory)
__device__ __forceinline__ void umma_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
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
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
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
// Barrier among the 8 epilogue warps only (the producer warps never join it).
__device__ __forceinline__ void epilogue_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

struct UmmaArgs {
  int32_t n_pseudo, group, n_q_heads, n_kv_heads;
  int32_t rows_total;        // G * N
  int32_t n_qgroups;         // ceil(rows_total / 256)
  int32_t has_lo;            // the query operand carries a low-order bf16 part
  int32_t lo_row_offset;     // rows between the hi and the lo copy in the query tensor
  float scale_log2e;
  const uint4* q;            // rotated queries, hi part: [B * H_q * N, 128] bf16 (sweep 1 reads it directly)
  float2* part;              // [n_chunks, H_kv, 2, n_qgroups * 256] (running max, sum) in base 2
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
__device__ __forceinline__ Work cta_work(const SeqTable& t, const ChunkTable& ct, const UmmaArgs& a, bool prompt_only) {
  Work w;
  const int chunk = blockIdx.x, kvh = blockIdx.y;
  w.b = find_segment(ct.cu_chunk, t.batch, chunk);
  w.L = t.prompt_len[w.b];
  const int n_tiles = (w.L + a.n_pseudo + kTileKeys - 1) / kTileKeys;
  w.t0 = (chunk - ct.cu_chunk[w.b]) * ct.chunk_tiles;
  int t1 = min(n_tiles, w.t0 + ct.chunk_tiles);
  if (prompt_only) t1 = min(t1, (w.L + kTileKeys - 1) / kTileKeys);   // tiles of synthetic keys give no score
  w.nt = t1 - w.t0;
  w.row_base = t.cu_rows[w.b];                                          // first cache row of the sequence
  w.qrow_base = (w.b * a.n_q_heads + kvh * a.group) * a.n_pseudo;       // first query row of this KV head
  return w;
}

// Running max / sum of exp over one 32-column piece of a sweep-1 accumulator row.
// lim: last visible column of the piece's tile for this thread's pseudo query (masked tiles).
template <bool kMasked>
__device__ __forceinline__ void row_stats_piece(const uint32_t* v, int col0, int lim, float c, float& m_raw, float& z) {
  float x[32];
#pragma unroll
  for (int e = 0; e < 32; ++e) {
    x[e] = __uint_as_float(v[e]);
    if (kMasked && col0 + e > lim) x[e] = -CUDART_INF_F;
  }
  float cmax = max3(x[0], x[1], x[2]);
#pragma unroll
  for (int e = 3; e < 31; e += 2) cmax = max3(cmax, x[e], x[e + 1]);
  cmax = fmaxf(cmax, x[31]);
  if (cmax > m_raw) {
    z *= ex2((m_raw - cmax) * c);
    m_raw = cmax;
  }
  if (!kMasked || m_raw > -CUDART_INF_F) {
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

// ============================================================================== sweep 1
__global__ void __launch_bounds__(kThreads, 1)
score_sweep1_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ SeqTable t,
                    const __grid_constant__ ChunkTable ct, const UmmaArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunk = blockIdx.x, kvh = blockIdx.y;
  const Work w = cta_work(t, ct, a, false);
  const int nt = w.nt, L = w.L, N = a.n_pseudo;
  if (nt <= 0) return;

  const uint32_t bar0 = sbase + Smem1::bars;
  auto k_full = [&](int s) { return bar0 + 8u * s; };
  auto k_empty = [&](int s) { return bar0 + 8u * (kStages1 + s); };
  auto acc_full = [&](int i) { return bar0 + 8u * (2 * kStages1 + i); };
  auto acc_empty = [&](int i) { return bar0 + 8u * (2 * kStages1 + 2 + i); };
  const uint32_t a_full = bar0 + 8u * (2 * kStages1 + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + Smem1::abort_flag);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + Smem1::tmem_ptr);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages1; ++s) { mbar_init(k_full(s), 1); mbar_init(k_empty(s), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(acc_full(i), 1); mbar_init(acc_empty(i), 4); }
    mbar_init(a_full, 8);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {                                              // tensor memory: all 512 columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(sbase + Smem1::tmem_ptr), "r"(kTmemCols) : "memory");
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
        for (int ti = 0; ti < nt; ++ti, ++li) {
          const int s = li % kStages1;
          if (li >= kStages1) ok = mbar_wait(k_empty(s), ((li / kStages1) - 1) & 1, abort_flag, a.status);
          if (!ok) break;
          mbar_expect_tx(k_full(s), kTileBytes);
          const int row = w.row_base + (w.t0 + ti) * kTileKeys;
          tma_load_3d(sbase + Smem1::k + s * kTileBytes, &tm_k, k_full(s), 0, row, kvh);
          tma_load_3d(sbase + Smem1::k + s * kTileBytes + kHalfBytesK, &tm_k, k_full(s), 64, row, kvh);
        }
      }
      if (!ok) {
        // aborting: let the copies already issued land before the CTA returns
        for (int back = 1; back <= kStages1 && back <= li; ++back) {
          const int l2 = li - back;
          const long long start = clock64();
          while (!mbar_try(k_full(l2 % kStages1), (l2 / kStages1) & 1) && clock64() - start < kWaitLimit) {}
        }
      }
    }
  } else if (warp == 1) {
    // ============================================================================= MMA issuer
    if (lane == 0) {
      int li = 0;
      uint32_t use0 = 0u, use1 = 0u;                            // jobs issued into each accumulator
      bool ok = true;
      const uint32_t idesc = umma_idesc(128, kTileKeys);
      for (int qg = 0; qg < a.n_qgroups && ok; ++qg) {
        const int rows_g = min(kGroupRows, a.rows_total - qg * kGroupRows);
        const int mb = (rows_g + 127) / 128;
        ok = mbar_wait(a_full, qg & 1, abort_flag, a.status);   // the group's queries are in tensor memory
        tc_fence_after();
        for (int ti = 0; ti < nt && ok; ++ti, ++li) {
          const int s = li % kStages1;
          ok = mbar_wait(k_full(s), (li / kStages1) & 1, abort_flag, a.status);
          if (!ok) break;
          const uint32_t kaddr = sbase + Smem1::k + s * kTileBytes;
          for (int m = 0; m < mb && ok; ++m) {
            // two blocks: block m -> accumulator m; one block: tiles alternate between the two
            const int buf = (mb == 2) ? m : (ti & 1);
            const uint32_t used = buf ? use1 : use0;
            if (used) ok = mbar_wait(acc_empty(buf), (used - 1) & 1, abort_flag, a.status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d = tmem_base + kAcc1 + buf * 128;
            uint32_t accum = 0;
            for (int part = 0; part < (a.has_lo ? 2 : 1); ++part) {
              const uint32_t a_addr = tmem_base + (2 * m + part) * kACols;
#pragma unroll
              for (int ks = 0; ks < 8; ++ks) {
                const int half = ks >> 2, kk = ks & 3;
                umma_ts(d, a_addr + ks * 8, umma_desc(kaddr + half * kHalfBytesK + kk * 32), idesc, accum);
                accum = 1;
              }
            }
            tc_commit(acc_full(buf));
            if (buf) ++use1; else ++use0;
          }
          tc_commit(k_empty(s));                                // the K stage is free once these MMAs retire
        }
      }
    }
  } else {
    // ============================================================================== epilogue
    const int eg = (warp - 2) >> 2;                             // epilogue group 0 / 1 = accumulator 0 / 1
    const int quad = warp & 3;                                  // TMEM lane quadrant of this warp
    const int r = quad * 32 + lane;                             // accumulator row of this thread
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float c = a.scale_log2e;
    uint32_t use = 0;                                           // jobs this group has taken from its accumulator
    bool ok = true;
    // (an aborting group still walks every query group: the other group waits for it at the barriers)
    for (int qg = 0; qg < a.n_qgroups; ++qg) {
      const int rows_g = min(kGroupRows, a.rows_total - qg * kGroupRows);
      const int mb = (rows_g + 127) / 128;
      // ---- this group's query block -> tensor memory (A operand: one row per lane, the 128
      // channels as 64 columns of bf16 pairs).  Rows past the KV head's G*N rows are zero.
      if (qg > 0) epilogue_sync();                              // every MMA that read the previous queries has retired
      if (eg < mb) {
        const int grow = qg * kGroupRows + eg * 128 + r;
        const bool valid = grow < a.rows_total;
        for (int part = 0; part < (a.has_lo ? 2 : 1); ++part) {
          const uint4* src = a.q + ((int64_t)part * a.lo_row_offset + w.qrow_base + grow) * 16;
#pragma unroll
          for (int hc = 0; hc < 2; ++hc) {
            uint32_t v[32];
#pragma unroll
            for (int x = 0; x < 8; ++x) {
              const uint4 u = valid ? __ldg(src + hc * 8 + x) : make_uint4(0u, 0u, 0u, 0u);
              v[4 * x] = u.x; v[4 * x + 1] = u.y; v[4 * x + 2] = u.z; v[4 * x + 3] = u.w;
            }
            tmem_st32(lane_addr + (2 * eg + part) * kACols + hc * 32, v);
          }
        }
        tmem_st_wait();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(a_full);

      float m_raw = -CUDART_INF_F, z = 0.f;                     // running max (raw dot product) and sum
      // pseudo-query index of this thread's row: block eg of a two-block group, else block 0
      const int my_blk = (mb == 2) ? eg : 0;
      const int i_q = (qg * kGroupRows + my_blk * 128 + r) % N;
      for (int ti = 0; ti < nt && ok; ++ti) {
        if (mb == 1 && (ti & 1) != eg) continue;                // one block: the groups take alternate tiles
        const int tile_base = (w.t0 + ti) * kTileKeys;
        const bool masked = tile_base + kTileKeys > L;          // holds synthetic (or foreign) rows
        ok = __all_sync(0xffffffffu, mbar_wait(acc_full(eg), use & 1, abort_flag, a.status));
        if (!ok) break;
        ++use;
        tc_fence_after();
        // key column `col` of this tile is visible to pseudo query i iff its position <= L + i
        const int lim = L + i_q - tile_base;                    // last visible column
        const uint32_t taddr = lane_addr + kAcc1 + eg * 128;
        uint32_t v[2][32];
        tmem_ld32(taddr, v[0]);
#pragma unroll
        for (int ch = 0; ch < kTileKeys / 32; ++ch) {
          tmem_ld_wait_for(v[ch & 1]);
          if (ch + 1 < kTileKeys / 32) tmem_ld32(taddr + (ch + 1) * 32, v[(ch + 1) & 1]);
          if (masked) row_stats_piece<true>(v[ch & 1], ch * 32, lim, c, m_raw, z);
          else row_stats_piece<false>(v[ch & 1], ch * 32, lim, c, m_raw, z);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty(eg));
      }
      // partials: slot eg of every row this group may own; neutral where it had no job
      float2* pbase = a.part + (((int64_t)chunk * a.n_kv_heads + kvh) * 2 + eg) * (a.n_qgroups * kGroupRows) +
                      qg * kGroupRows;
      for (int m = 0; m < mb; ++m) {
        const bool mine = (mb == 1) || (m == eg);               // with 2 blocks, group e takes block e
        if (qg * kGroupRows + m * 128 + r < a.rows_total)
          pbase[m * 128 + r] = mine ? make_float2(m_raw * c, z) : make_float2(-CUDART_INF_F, 0.f);
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

// ============================================================================== sweep 2
__global__ void __launch_bounds__(kThreads, 1)
score_sweep2_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_q,
                    const __grid_constant__ SeqTable t, const __grid_constant__ ChunkTable ct, const UmmaArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunk = blockIdx.x, kvh = blockIdx.y;
  const Work w = cta_work(t, ct, a, true);
  const int nt = w.nt, L = w.L, b = w.b;
  if (nt <= 0) return;

  const uint32_t bar0 = sbase + Smem2::bars;
  auto k_full = [&](int s) { return bar0 + 8u * s; };
  auto k_empty = [&](int s) { return bar0 + 8u * (kStages2 + s); };
  auto acc_full = [&](int i) { return bar0 + 8u * (2 * kStages2 + i); };
  auto acc_empty = [&](int i) { return bar0 + 8u * (2 * kStages2 + 2 + i); };
  const uint32_t q_full = bar0 + 8u * (2 * kStages2 + 4), q_empty = bar0 + 8u * (2 * kStages2 + 5);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + Smem2::abort_flag);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + Smem2::tmem_ptr);
  float* lse_s = reinterpret_cast<float*>(smem + Smem2::lse);   // [256] base-2 lse of the resident query group

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages2; ++s) { mbar_init(k_full(s), 1); mbar_init(k_empty(s), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(acc_full(i), 1); mbar_init(acc_empty(i), 4); }
    mbar_init(q_full, 1);
    mbar_init(q_empty, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {                                              // tensor memory: all 512 columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(sbase + Smem2::tmem_ptr), "r"(kTmemCols) : "memory");
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
              tma_load_2d(sbase + (part ? Smem2::q_lo : Smem2::q_hi) + half * kHalfBytesQ + m * 128 * 128, &tm_q, q_full,
                          half * 64, part * a.lo_row_offset + w.qrow_base + qg * kGroupRows + m * 128);
        for (int ti = 0; ti < nt; ++ti, ++li) {
          const int s = li % kStages2;
          if (li >= kStages2) ok = mbar_wait(k_empty(s), ((li / kStages2) - 1) & 1, abort_flag, a.status);
          if (!ok) break;
          mbar_expect_tx(k_full(s), kTileBytes);
          const int row = w.row_base + (w.t0 + ti) * kTileKeys;
          tma_load_3d(sbase + Smem2::k + s * kTileBytes, &tm_k, k_full(s), 0, row, kvh);
          tma_load_3d(sbase + Smem2::k + s * kTileBytes + kHalfBytesK, &tm_k, k_full(s), 64, row, kvh);
        }
      }
      if (!ok) {
        // aborting: let the copies already issued land before the CTA returns
        for (int back = 1; back <= kStages2 && back <= li; ++back) {
          const int l2 = li - back;
          const long long start = clock64();
          while (!mbar_try(k_full(l2 % kStages2), (l2 / kStages2) & 1) && clock64() - start < kWaitLimit) {}
        }
      }
    }
  } else if (warp == 1) {
    // ============================================================================= MMA issuer
    if (lane == 0) {
      int job = 0;                                              // = K tiles consumed: one job per tile
      bool ok = true;
      for (int qg = 0; qg < a.n_qgroups && ok; ++qg) {
        const int rows_g = min(kGroupRows, a.rows_total - qg * kGroupRows);
        const uint32_t idesc = umma_idesc(128, (rows_g + 15) & ~15);   // only the query columns that exist
        ok = mbar_wait(q_full, qg & 1, abort_flag, a.status);
        for (int ti = 0; ti < nt && ok; ++ti, ++job) {
          const int s = job % kStages2, buf = job & 1;
          ok = mbar_wait(k_full(s), (job / kStages2) & 1, abort_flag, a.status);
          if (ok && job >= 2) ok = mbar_wait(acc_empty(buf), ((job >> 1) - 1) & 1, abort_flag, a.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t kaddr = sbase + Smem2::k + s * kTileBytes;
          const uint32_t d = tmem_base + buf * 256;
          uint32_t accum = 0;
          for (int part = 0; part < (a.has_lo ? 2 : 1); ++part) {
            const uint32_t qaddr = sbase + (part ? Smem2::q_lo : Smem2::q_hi);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const int half = ks >> 2, kk = ks & 3;
              umma_ss(d, umma_desc(kaddr + half * kHalfBytesK + kk * 32), umma_desc(qaddr + half * kHalfBytesQ + kk * 32),
                      idesc, accum);
              accum = 1;
            }
          }
          tc_commit(acc_full(buf));
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
    for (int qg = 0; qg < a.n_qgroups; ++qg) {
      const int rows_g = min(kGroupRows, a.rows_total - qg * kGroupRows);
      // ---- base-2 log-sum-exp of the group's rows: thread (eg, r) merges the per-chunk
      // partials of row eg*128 + r in a fixed order, or converts the caller's value
      if (qg > 0) epilogue_sync();                              // the previous group's values are no longer read
      {
        const int row = eg * 128 + r, grow = qg * kGroupRows + row;
        float l2 = 0.f;
        if (grow < a.rows_total) {
          if (a.lse_in) {
            l2 = a.lse_in[w.qrow_base + grow] * 1.4426950408889634f;
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
          if (a.lse_out && chunk == ct.cu_chunk[b]) a.lse_out[w.qrow_base + grow] = l2 * 0.6931471805599453f;
        }
        lse_s[row] = l2;
      }
      epilogue_sync();
      // Tile ti always goes to group ti & 1, so one thread owns a key's score across all
      // query groups and accumulates it in program order.
      const int nch = (rows_g + 31) >> 5;                       // 32-column pieces of a job
      for (int ti = 0; ti < nt && ok; ++ti, ++job) {
        if ((ti & 1) != eg) continue;
        const int buf = job & 1;
        ok = __all_sync(0xffffffffu, mbar_wait(acc_full(buf), (job >> 1) & 1, abort_flag, a.status));
        if (!ok) break;
        tc_fence_after();
        const uint32_t taddr = lane_addr + buf * 256;
        float sum0 = 0.f, sum1 = 0.f;
        uint32_t v[2][32];
        tmem_ld32(taddr, v[0]);
#pragma unroll
        for (int ch = 0; ch < kGroupRows / 32; ++ch) {
          if (ch < nch) {
            tmem_ld_wait_for(v[ch & 1]);
            if (ch + 1 < nch) tmem_ld32(taddr + (ch + 1) * 32, v[(ch + 1) & 1]);
            const int valid = rows_g - ch * 32;                 // >= 32 except in the last piece
            if (valid >= 32) {
#pragma unroll
              for (int e = 0; e < 32; e += 4) {
                const float4 l4 = *reinterpret_cast<const float4*>(lse_s + ch * 32 + e);
                sum0 += ex2(fmaf(__uint_as_float(v[ch & 1][e]), c, -l4.x));
                sum1 += ex2(fmaf(__uint_as_float(v[ch & 1][e + 1]), c, -l4.y));
                sum0 += ex2(fmaf(__uint_as_float(v[ch & 1][e + 2]), c, -l4.z));
                sum1 += ex2(fmaf(__uint_as_float(v[ch & 1][e + 3]), c, -l4.w));
              }
            } else {
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (e < valid) sum0 += ex2(fmaf(__uint_as_float(v[ch & 1][e]), c, -lse_s[ch * 32 + e]));
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty(buf));
        const int j = (w.t0 + ti) * kTileKeys + r;              // sequence-local key position
        if (j < L) {
          float* out = a.scores + (int64_t)kvh * a.score_stride + t.cu_prompt[b] + j;
          const float sum = sum0 + sum1;
          *out = (qg == 0) ? sum : *out + sum;
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
  int max_tiles = 0;
  for (int b = 0; b < t.batch; ++b) {
    const int tiles = (t.prompt_len[b] + n_pseudo + kTileKeys - 1) / kTileKeys;
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
  plan->q_hi = q_hi;
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
  a.q = static_cast<const uint4*>(plan.q_hi);
  a.part = part;
  a.lse_in = lse_in;
  a.lse_out = lse_out;
  a.scores = scores;
  a.score_stride = score_stride;
  a.status = status;

  cudaError_t e;
  if ((e = cudaFuncSetAttribute(score_sweep1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes1)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(score_sweep2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes2)) != cudaSuccess) return e;
  const dim3 grid(ct.n_chunks, dm.n_kv_heads);
  if (lse_in == nullptr) {
    log->begin(kKindSweep1, s);
    score_sweep1_kernel<<<grid, kThreads, kSmemBytes1, s>>>(plan.tm_k, t, ct, a);
    log->end(s);
  }
  log->begin(kKindSweep2, s);
  score_sweep2_kernel<<<grid, kThreads, kSmemBytes2, s>>>(plan.tm_k, plan.tm_q, t, ct, a);
  log->end(s);
  return cudaGetLastError();
}

}  // namespace dapq
