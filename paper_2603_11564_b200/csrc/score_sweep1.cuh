// Sweep 1 of the tensor-core scorer: per pseudo query, the running maximum and the sum of
// exponentials of its logits over the CTA's chunk of keys (Appendix C, Step 1: s_j = q k_j /
// sqrt(d_k); the softmax normaliser of Section 4.2, Eq. 4 is built from these partials).
//
//   D[query, key] = Q_blk K_tile^T, queries on tensor-memory lanes, 192 keys per tile.
// A job is one [128 queries x 192 keys] accumulator; the two query blocks of a group own one
// accumulator each, so the MMAs of one block run while the other block's accumulator is read
// (a group of one block alternates between the two accumulators from tile to tile).
// All four epilogue groups work on every job, 48 key columns each: thread (group g, row r) keeps
// the statistics of query row r over the columns of its group; at the end of a chunk the four
// groups fold their statistics together through shared memory into the row's per-chunk partial.
// Sixteen epilogue warps (four per scheduler) hide the latency of the tensor-memory loads and of
// the hand-offs, so each reads its columns in plain 16-column pieces.
#pragma once
#include "score_umma_common.cuh"

namespace dapq {
namespace umma {

// Running max / sum of exp over one 16-column piece of an accumulator row.
// lim: last visible column of the piece's tile for this thread's pseudo query (masked tiles).
template <bool kMasked>
__device__ __forceinline__ void row_stats_piece(const uint32_t* v, int col0, int lim, float c, float& m_raw, float& z) {
  float x[16];
#pragma unroll
  for (int e = 0; e < 16; ++e) {
    x[e] = __uint_as_float(v[e]);
    if (kMasked && col0 + e > lim) x[e] = -CUDART_INF_F;
  }
  float cmax = max3(x[0], x[1], x[2]);
#pragma unroll
  for (int e = 3; e < 15; e += 2) cmax = max3(cmax, x[e], x[e + 1]);
  cmax = fmaxf(cmax, x[15]);
  if (cmax > m_raw) {
    z *= ex2((m_raw - cmax) * c);
    m_raw = cmax;
  }
  if (!kMasked || m_raw > -CUDART_INF_F) {
    const float neg = -m_raw * c;
    // pairs of columns on the packed fp32 pipe; 2^x by MUFU or, for the pairs of kPolyPairMask, by polynomial
    const float2 c2 = make_float2(c, c), neg2 = make_float2(neg, neg);
    float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll
    for (int e = 0; e < 16; e += 4) {
      const float2 x0 = __ffma2_rn(make_float2(x[e], x[e + 1]), c2, neg2);
      const float2 x1 = __ffma2_rn(make_float2(x[e + 2], x[e + 3]), c2, neg2);
      acc0 = __fadd2_rn(acc0, ((kPolyPairMask >> (e / 2)) & 1u) ? ex2_pair_poly(x0) : ex2_pair_mufu(x0));
      acc1 = __fadd2_rn(acc1, ((kPolyPairMask >> (e / 2 + 1)) & 1u) ? ex2_pair_poly(x1) : ex2_pair_mufu(x1));
    }
    z += (acc0.x + acc0.y) + (acc1.x + acc1.y);
  }
}

// (max, sum of exp2) of two disjoint sets of logits -> of their union.
__device__ __forceinline__ float2 merge_stats(float2 a, float2 b) {
  const float m = fmaxf(a.x, b.x);
  if (m == -CUDART_INF_F) return make_float2(m, 0.f);
  return make_float2(m, a.y * exp2f(a.x - m) + b.y * exp2f(b.x - m));
}

// This group's 48 columns of one accumulator, in three 16-column pieces; `release` gives the accumulator
// back once the last piece is in registers.
template <class Release>
__device__ __forceinline__ void row_stats_job(uint32_t taddr, int col0, bool masked, int lim, float c, float& m_raw,
                                              float& z, Release release) {
  constexpr int kPieces = kTile1 / kEpiGroups / 16;
#pragma unroll
  for (int ch = 0; ch < kPieces; ++ch) {
    uint32_t v[16];
    tmem_ld16(taddr + ch * 16, v);
    tmem_ld_wait_for16(v);
    if (ch == kPieces - 1) release();
    if (masked) row_stats_piece<true>(v, col0 + ch * 16, lim, c, m_raw, z);
    else row_stats_piece<false>(v, col0 + ch * 16, lim, c, m_raw, z);
  }
}

template <bool kCompact>
__global__ void __launch_bounds__(kThreads, 1)
score_sweep1_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_q,
                    const __grid_constant__ SeqTable t, const __grid_constant__ ChunkTable ct, const UmmaArgs a) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  if (sbase & 1023u) {                                          // (uniform over the CTA: nothing has been set up yet)
    if (threadIdx.x == 0) atomicOr(a.status, kStatusSmemAlign);
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  using G = Geo<kCompact>;
  constexpr int kStages1 = G::kStages1;
  const int chunk = blockIdx.x, kvh = blockIdx.y;
  const Work w = cta_work(t, ct, a, kTile1, true);
  const int nt = w.nt, L = w.L, N = a.n_pseudo;
  if (nt <= 0) return;
  const Bars bars{sbase + Smem::bars};
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + Smem::abort_flag);
  const uint32_t tmem_base = cta_prologue(smem, sbase, bars, kStages1, 2);

  if (warp == 0) {
    if (lane == 0)
      tma_producer<G, kTile1, kStages1, kStageBytes1, kHalfBytes1>(&tm_k, &tm_q, w, a, sbase, bars, kvh, abort_flag);
  } else if (warp == 1) {
    // ============================================================================= MMA issuer
    if (lane == 0) {
      int li = 0, n_done = 0;
      uint32_t use0 = 0u, use1 = 0u;                            // jobs issued into each accumulator
      bool ok = true;
      const uint32_t idesc = umma_idesc(128, kTile1);
      const uint64_t qd_hi = umma_desc(sbase + G::q_hi), qd_lo = umma_desc(sbase + G::q_lo);
      for (int qg = 0; qg < a.n_qgroups && ok; ++qg) {
        const int rows_g = min(G::kRows, a.rows_total - qg * G::kRows);
        const int mb = (rows_g + 127) / 128;
        ok = mbar_wait_limit(bars.q_full(), qg & 1, abort_flag, a.status, a.wait_limit);
        for (int ti = 0; ti < nt && ok; ++ti, ++li) {
          const int s = li % kStages1;
          ok = mbar_wait_limit(bars.k_full(s), (li / kStages1) & 1, abort_flag, a.status, a.wait_limit);
          if (!ok) break;
          const uint64_t kd = umma_desc(sbase + G::k + s * kStageBytes1);
          for (int m = 0; m < mb && ok; ++m) {
            // two blocks: block m -> accumulator m; one block: tiles alternate between the two
            const int buf = (mb == 2) ? m : (ti & 1);
            const uint32_t used = buf ? use1 : use0;
            if (used) ok = mbar_wait_limit(bars.acc_empty(buf), (used - 1) & 1, abort_flag, a.status, a.wait_limit);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d = tmem_base + buf * kTile1;
            const uint64_t qh = desc_advance(qd_hi, m * 128 * 128), ql = desc_advance(qd_lo, m * 128 * 128);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const int half = ks >> 2, kk = ks & 3;
              umma_ss(d, desc_advance(qh, half * G::kHalfBytesQ + kk * 32), desc_advance(kd, half * kHalfBytes1 + kk * 32),
                      idesc, ks ? 1u : 0u);
            }
            if (a.has_lo) {
#pragma unroll
              for (int ks = 0; ks < 8; ++ks) {
                const int half = ks >> 2, kk = ks & 3;
                umma_ss(d, desc_advance(ql, half * G::kHalfBytesQ + kk * 32), desc_advance(kd, half * kHalfBytes1 + kk * 32),
                        idesc, 1u);
              }
            }
            tc_commit(bars.acc_full(buf));
            if (buf) ++use1; else ++use0;
          }
          tc_commit(bars.k_empty(s));                           // the K stage is free once these MMAs retire
        }
        tc_commit(bars.q_empty());
        ++n_done;
      }
      mma_drain(bars, n_done, n_done < a.n_qgroups);
    }
  } else {
    // ============================================================================== epilogue
    const int eg = (warp - 2) >> 2;                             // epilogue group 0 .. 3: key columns 48 eg .. 48 eg + 47
    const int quad = warp & 3;                                  // TMEM lane quadrant of this warp
    const int r = quad * 32 + lane;                             // accumulator row of this thread
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float c = a.scale_log2e;
    const int col0 = eg * (kTile1 / kEpiGroups);
    uint32_t use0 = 0u, use1 = 0u;                              // jobs taken from each accumulator
    float2* stat = reinterpret_cast<float2*>(smem + Smem::lse);  // [256] (max, sum) of the rows on their way through the groups
    bool ok = true;
    // (an aborting warp still walks every query group: the others wait for it at the barriers)
    for (int qg = 0; qg < a.n_qgroups; ++qg) {
      const int rows_g = min(G::kRows, a.rows_total - qg * G::kRows);
      const int mb = (rows_g + 127) / 128;
      // running max (raw dot product) and sum of this thread's row of block 0 / block 1
      float m_raw0 = -CUDART_INF_F, z0 = 0.f, m_raw1 = -CUDART_INF_F, z1 = 0.f;
      const int i_q0 = (qg * G::kRows + r) % N, i_q1 = (qg * G::kRows + 128 + r) % N;   // pseudo-query indices
      for (int ti = 0; ti < nt && ok; ++ti) {
        const int tile_base = (w.t0 + ti) * kTile1;
        const bool masked = tile_base + kTile1 > L;             // holds synthetic (or foreign) rows
        for (int m = 0; m < mb && ok; ++m) {
          const int buf = (mb == 2) ? m : (ti & 1);
          const uint32_t used = buf ? use1 : use0;
          ok = __all_sync(0xffffffffu, mbar_wait_limit(bars.acc_full(buf), used & 1, abort_flag, a.status, a.wait_limit));
          if (!ok) break;
          if (buf) ++use1; else ++use0;
          tc_fence_after();
          const uint32_t taddr = lane_addr + buf * kTile1 + col0;
          auto release = [&] {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bars.acc_empty(buf));
          };
          // key column `col` of this tile is visible to pseudo query i iff its position <= L + i
          if (m == 0) row_stats_job(taddr, col0, masked, L + i_q0 - tile_base, c, m_raw0, z0, release);
          else row_stats_job(taddr, col0, masked, L + i_q1 - tile_base, c, m_raw1, z1, release);
        }
      }
      // The four groups hold the statistics of the same rows over different key columns: group 3 puts its
      // pair into shared memory, groups 2 and 1 fold theirs in, group 0 folds last and stores the chunk's
      // partials (a fixed order, so the result does not depend on timing).
      float2 s0 = make_float2(m_raw0 * c, z0), s1 = make_float2(m_raw1 * c, z1);
      if (qg > 0) epilogue_sync();                              // group 0 has read the round before
#pragma unroll
      for (int g = kEpiGroups - 1; g >= 0; --g) {
        if (eg == g) {
          if (g < kEpiGroups - 1) {
            s0 = merge_stats(s0, stat[r]);
            s1 = merge_stats(s1, stat[128 + r]);
          }
          if (g > 0) {
            stat[r] = s0;
            stat[128 + r] = s1;
          }
        }
        if (g > 0) epilogue_sync();
      }
      if (eg == 0) {
        float2* pbase = a.part + ((int64_t)chunk * a.n_kv_heads + kvh) * a.rows_pad + qg * G::kRows;
        if (qg * G::kRows + r < a.rows_total) pbase[r] = s0;
        if (mb == 2 && qg * G::kRows + 128 + r < a.rows_total) pbase[128 + r] = s1;
      }
    }
  }
  cta_epilogue(tmem_base);
}

}  // namespace umma
}  // namespace dapq
