// Sweep 1 of the tensor-core scorer: per pseudo query, the running maximum and the sum of
// exponentials of its logits over the CTA's chunk of keys (Appendix C, Step 1: s_j = q k_j /
// sqrt(d_k); the softmax normaliser of Section 4.2, Eq. 4 is built from these partials).
//
//   D[query, key] = Q_blk K_tile^T, queries on tensor-memory lanes, 192 keys per tile.
// CTA = (chunk of K tiles, query group, KV head), as in sweep 2.  A job is one [128 queries x 192 keys]
// accumulator; the two query blocks of a group own one accumulator each, so the MMAs of one block run
// while the other block's accumulator is read (a group of one block alternates between the two
// accumulators from tile to tile).  All four epilogue groups work on every job, 48 key columns each:
// thread (group g, row r) reads its 48 columns in one go, gives the accumulator back, and folds them
// into the statistics of query row r with one maximum and at most one rescaling per job; no warp waits
// for another one until the end of the chunk, where the four groups fold their statistics together
// through shared memory into the row's per-chunk partial.
#pragma once
#include "score_qg_common.cuh"

namespace dapq {
namespace qg {

constexpr int kCols1 = kTile1 / kEpiGroups;    // key columns of a job per epilogue group
// Column pairs of a job that take the polynomial exp2 when the sums run without a maximum: none.  That path
// has so few instructions per element left that it runs at the pace of the MUFU pipe either way (measured on
// the Llama-3-70B shape: 0, 1/8 and 1/4 of the pairs on the polynomial are within 2 % of one another, in
// both directions from one GPU to the next), so it keeps the simplest form.
#ifndef DAPQ_POLY_PAIR_MASK_SUM
#define DAPQ_POLY_PAIR_MASK_SUM 0x0000u
#endif
constexpr uint32_t kPolyPairMaskSum = DAPQ_POLY_PAIR_MASK_SUM;

// Running max / sum of exp over this thread's 48 columns of an accumulator row.
// lim: last visible column of the tile for this thread's pseudo query (masked tiles only).
template <bool kMasked>
__device__ __forceinline__ void row_stats_cols(uint32_t* v, int col0, int lim, float c, float& m_raw, float& z) {
  float* x = reinterpret_cast<float*>(v);
  if (kMasked) {
#pragma unroll
    for (int e = 0; e < kCols1; ++e)
      if (col0 + e > lim) x[e] = -CUDART_INF_F;
  }
  float m0 = max3(x[0], x[1], x[2]), m1 = max3(x[3], x[4], x[5]), m2 = max3(x[6], x[7], x[8]), m3 = max3(x[9], x[10], x[11]);
#pragma unroll
  for (int e = 12; e + 8 <= kCols1; e += 8) {
    m0 = max3(m0, x[e], x[e + 1]);
    m1 = max3(m1, x[e + 2], x[e + 3]);
    m2 = max3(m2, x[e + 4], x[e + 5]);
    m3 = max3(m3, x[e + 6], x[e + 7]);
  }
  static_assert((kCols1 - 12) % 8 == 4 || (kCols1 - 12) % 8 == 0, "column count does not fit the maximum tree");
  float cmax;
  if ((kCols1 - 12) % 8 == 4) {
    // the loop above ran over [12, 12 + 8 n): the last four columns are still open
    cmax = fmaxf(max3(m0, m1, x[kCols1 - 4]), max3(m2, m3, x[kCols1 - 3]));
    cmax = max3(cmax, x[kCols1 - 2], x[kCols1 - 1]);
  } else {
    cmax = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
  }
  if (cmax > m_raw) {
    z *= ex2((m_raw - cmax) * c);                               // ex2(-inf) = 0 on the first job
    m_raw = cmax;
  }
  if (!kMasked || m_raw > -CUDART_INF_F) {
    const float neg = -m_raw * c;
    // pairs of columns on the packed fp32 pipe; 2^x by MUFU or, for the pairs of kPolyPairMask, by polynomial
    const float2 c2 = make_float2(c, c), neg2 = make_float2(neg, neg);
    float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll
    for (int e = 0; e < kCols1; e += 4) {
      const float2 x0 = __ffma2_rn(make_float2(x[e], x[e + 1]), c2, neg2);
      const float2 x1 = __ffma2_rn(make_float2(x[e + 2], x[e + 3]), c2, neg2);
      acc0 = __fadd2_rn(acc0, ((kPolyPairMask >> ((e / 2) & 15)) & 1u) ? ex2_pair_poly(x0) : ex2_pair_mufu(x0));
      acc1 = __fadd2_rn(acc1, ((kPolyPairMask >> ((e / 2 + 1) & 15)) & 1u) ? ex2_pair_poly(x1) : ex2_pair_mufu(x1));
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

// Row statistics without a running maximum.  With the library's own fp16 queries every job's MMAs end with
// one more k-step that subtracts a per-row reference logit r (the row's logit against the first key of its
// sequence, written by the rotation kernel), so the accumulator holds x = logit - r and a job is just
// z += sum 2^x: no maximum, no rescaling, no subtraction.  The sum of a row is kept as z * 2^m with m = r
// at first.  The result stays exact for every input: a job whose sum leaves the float range (a key more
// than ~2^127 above the reference) is redone from its registers with its own maximum and merged, which
// moves m; once m is far from r every job takes that careful path.  Logits far BELOW r only underflow
// against a term, the reference key's own, that is part of the same row's total.
struct RowSum {
  float r, m, z, sc;                                            // reference, base of z, sum, 2^(r - m)
  __device__ __forceinline__ void init(float ref) { r = m = ref; z = 0.f; sc = 1.f; }
};
template <bool kMasked>
__device__ __forceinline__ void row_sum_cols(uint32_t* v, int col0, int lim, RowSum& st) {
  float* x = reinterpret_cast<float*>(v);
  if (kMasked) {
#pragma unroll
    for (int e = 0; e < kCols1; ++e)
      if (col0 + e > lim) x[e] = -CUDART_INF_F;
  }
  if (st.m - st.r < 100.f) {
    float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll
    for (int e = 0; e < kCols1; e += 4) {
      const float2 x0 = make_float2(x[e], x[e + 1]), x1 = make_float2(x[e + 2], x[e + 3]);
      acc0 = __fadd2_rn(acc0, ((kPolyPairMaskSum >> ((e / 2) & 15)) & 1u) ? ex2_pair_poly<true>(x0) : ex2_pair_mufu(x0));
      acc1 = __fadd2_rn(acc1, ((kPolyPairMaskSum >> ((e / 2 + 1) & 15)) & 1u) ? ex2_pair_poly<true>(x1) : ex2_pair_mufu(x1));
    }
    const float zj = (acc0.x + acc0.y) + (acc1.x + acc1.y);
    if (zj < 1e37f) {                                           // (false for inf and NaN too)
      st.z = fmaf(zj, st.sc, st.z);
      if (st.z > 1e30f) {                                       // keep z well inside the float range
        st.m += 64.f;
        st.z *= 5.421010862427522e-20f;                         // 2^-64
        st.sc *= 5.421010862427522e-20f;
      }
      return;
    }
  }
  // careful path: this job's own maximum and sum (relative to r), merged into the row's
  float ml = -CUDART_INF_F, zl = 0.f;
  row_stats_cols<kMasked>(v, col0, lim, 1.f, ml, zl);
  if (ml > -CUDART_INF_F) {
    const float2 mg = merge_stats(make_float2(st.m, st.z), make_float2(st.r + ml, zl));
    st.m = mg.x;
    st.z = mg.y;
    st.sc = exp2f(st.r - st.m);
  }
}

template <bool kConvert>
__global__ void __launch_bounds__(kThreads1, 1)
rowstat_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_q,
               const __grid_constant__ SeqTable t, const __grid_constant__ ChunkTable ct, const Args a) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  if (sbase & 1023u) {                                          // (uniform over the CTA: nothing has been set up yet)
    if (threadIdx.x == 0) atomicOr(a.status, kStatusSmemAlign);
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  using T = TileGeo<kTile1>;
  constexpr bool kFold = kConvert;                              // the library's own fp16 queries come with reference logits
  const int kvh = blockIdx.y;
  const Work w = cta_work(t, ct, a, kTile1, true);
  const int nt = w.nt, L = w.L, N = a.n_pseudo, mb = w.mb;
  if (nt <= 0) return;
  const Bars bars{sbase + Smem::bars};
  const Waiter wt{reinterpret_cast<volatile int*>(smem + Smem::abort_flag), a.status, a.wait_limit};
  // With reference logits: the epilogue threads ask for theirs first of all (the rotation kernel, the kernel before
  // this one, wrote them), before the CTA's copies of keys and queries crowd the memory system: row te of the
  // [256 x 16] operand, and the thread's own two accumulator rows.
  float ref_slab = 0.f, ref_r0 = 0.f, ref_r1 = 0.f;
  if (kFold && warp >= kFirstEpiWarp) {
    pdl_wait();
    const float* ref = a.ref + w.qrow_base + w.qgrp * a.rows_g;
    const int te = (warp - kFirstEpiWarp) * 32 + lane, r_ = (warp & 3) * 32 + lane;
    if (te < w.rows) ref_slab = __ldg(ref + te);
    if (r_ < w.rows) ref_r0 = __ldg(ref + r_);
    if (128 + r_ < w.rows) ref_r1 = __ldg(ref + 128 + r_);
  }
  // (the keys are nobody's output in this stream; the queries are the rotation kernel's, the kernel before)
  const uint32_t tmem_base = cta_prologue(smem, sbase, bars, [&] {
    if (a.early_loads) tma_first<kTile1, false>(&tm_k, &tm_q, w, a, sbase, bars, kvh);
  });
  const uint32_t q_half = (uint32_t)mb * 128u * 128u;           // bytes of one 64-channel half of the query group
  const int S = a.n_stages;

  if (warp == 0) {
    if (lane == 0) {
      if (!a.early_loads) tma_first<kTile1, false>(&tm_k, &tm_q, w, a, sbase, bars, kvh);
      tma_producer<kTile1, true, false>(&tm_k, &tm_q, w, a, sbase, bars, kvh, wt);
    }
  } else if (warp == 1) {
    // ============================================================================= MMA issuer
    if (lane == 0) {
      uint32_t use0 = 0u, use1 = 0u;                            // jobs issued into each accumulator
      bool ok = wt.wait(bars.q_full(), 0);
      if (ok && kFold) ok = wt.wait(bars.lse_ready(), 0);
      const uint32_t idesc = kConvert ? umma_idesc_f16(128, kTile1) : umma_idesc(128, kTile1);
      const uint64_t qd = umma_desc(sbase);
      const uint64_t ref_d = umma_desc_rows32(sbase + kRefSlab), ones_d = umma_desc_rows32(sbase + Smem::exch);
      const uint32_t ring = sbase + 2 * q_half;
      Ring rs(S);
      for (int ti = 0; ti < nt && ok; ++ti, rs.next()) {
        const int s = rs.i;
        ok = wt.wait(kConvert ? bars.k_conv(s) : bars.k_full(s), rs.phase);
        if (!ok) break;
        const uint64_t kd = umma_desc(ring + s * T::kStage);
        for (int m = 0; m < mb && ok; ++m) {
          // two blocks: block m -> accumulator m; one block: tiles alternate between the two
          const int buf = (mb == 2) ? m : (ti & 1);
          const uint32_t used = buf ? use1 : use0;
          if (used) ok = wt.wait(bars.acc_empty(buf), (used - 1) & 1);
          if (!ok) break;
          tc_fence_after();
          const uint32_t d = tmem_base + buf * kTile1;
          const uint64_t qm = desc_advance(qd, m * 128 * 128);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const int half = ks >> 2, kk = ks & 3;
            umma_ss(d, desc_advance(qm, half * q_half + kk * 32), desc_advance(kd, half * T::kHalf + kk * 32), idesc, ks ? 1u : 0u);
          }
          if (kFold) umma_ss(d, desc_advance(ref_d, m * 128 * 32), ones_d, idesc, 1u);   // D[i, key] += (-r_i) * 1
          tc_commit(bars.acc_full(buf));
          if (buf) ++use1; else ++use0;
        }
        tc_commit(bars.k_empty(s));                             // the K stage is free once these MMAs retire
      }
      mma_drain(bars);
    }
  } else if (warp < kFirstEpiWarp) {
    if (kConvert) convert_tiles<kTile1>(w, a, sbase, bars, warp - 2, wt);
  } else {
    // ============================================================================== epilogue
    const int eg = (warp - kFirstEpiWarp) >> 2;                 // epilogue group 0 .. 3: key columns 48 eg .. 48 eg + 47
    const int quad = warp & 3;                                  // TMEM lane quadrant of this warp
    const int r = quad * 32 + lane;                             // accumulator row of this thread
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float c = a.scale_log2e;
    const int col0 = eg * kCols1;
    uint32_t use0 = 0u, use1 = 0u;                              // jobs taken from each accumulator
    float2* stat = reinterpret_cast<float2*>(smem + Smem::lse);  // [256] (max, sum) of the rows on their way through the groups
    bool ok = true;
    // running max (raw dot product) and sum of this thread's row of block 0 / block 1
    float m_raw0 = -CUDART_INF_F, z0 = 0.f, m_raw1 = -CUDART_INF_F, z1 = 0.f;
    RowSum rs0, rs1;                                            // ... or, with reference logits, the rows' sums
    const int i_q0 = (w.qgrp * a.rows_g + r) % N, i_q1 = (w.qgrp * a.rows_g + 128 + r) % N;   // pseudo-query indices
    if (kFold) {
      // The [256 x 16] operand: row i holds -r_i as an fp16 pair in channels 0 and 1 (zeros elsewhere, also
      // for rows beyond the group); the operand of ones carries its two ones in BOTH 16-byte halves of every
      // row, so whichever way the 32-byte swizzle orders the halves, the k-step adds exactly hi + lo.
      const int te = (warp - kFirstEpiWarp) * 32 + lane;        // 0 .. 511
      auto split = [&](int row, float ref_val, uint32_t& pair) -> float {   // the reference as the MMAs will see it
        if (row >= w.rows) { pair = 0u; return 0.f; }
        const float l = -ref_val;
        const __half hi = __float2half_rn(l), lo = __float2half_rn(l - __half2float(hi));
        pair = (uint32_t)__half_as_ushort(hi) | ((uint32_t)__half_as_ushort(lo) << 16);
        return -(__half2float(hi) + __half2float(lo));
      };
      if (te < kGroupRows) {
        uint32_t pair;
        split(te, ref_slab, pair);
        const uint32_t dst = sbase + kRefSlab + (te >> 3) * 256 + (te & 7) * 32;
        sts128(dst, make_uint4(pair, 0u, 0u, 0u));
        sts128(dst + 16, make_uint4(0u, 0u, 0u, 0u));
      }
      if (te < kOnes1SlabBytes / 16) sts128(sbase + Smem::exch + te * 16, make_uint4(0x3c003c00u, 0u, 0u, 0u));
      fence_proxy_async();                                      // the MMAs read both operands through the async proxy
      uint32_t unused;
      rs0.init(split(r, ref_r0, unused));
      rs1.init(split(128 + r, ref_r1, unused));
      epilogue_sync();
      if (warp == kFirstEpiWarp && lane == 0) mbar_arrive(bars.lse_ready());
    }
    for (int ti = 0; ti < nt && ok; ++ti) {
      const int tile_base = (w.t0 + ti) * kTile1;
      const bool masked = tile_base + kTile1 > L;               // holds synthetic (or foreign) rows
      for (int m = 0; m < mb && ok; ++m) {
        const int buf = (mb == 2) ? m : (ti & 1);
        const uint32_t used = buf ? use1 : use0;
        ok = __all_sync(0xffffffffu, wt.wait(bars.acc_full(buf), used & 1));
        if (!ok) break;
        if (buf) ++use1; else ++use0;
        tc_fence_after();
        const uint32_t taddr = lane_addr + buf * kTile1 + col0;
        uint32_t v[kCols1];
        tmem_ld16(taddr, v);
        tmem_ld16(taddr + 16, v + 16);
        tmem_ld16(taddr + 32, v + 32);
        tmem_ld_wait_for(v);
        tmem_ld_wait_for16(v + 32);
        // the accumulator goes back to the MMA issuer as soon as its columns are in registers
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bars.acc_empty(buf));
        // key column `col` of this tile is visible to pseudo query i iff its position <= L + i
        if (kFold) {
          if (m == 0) {
            if (masked) row_sum_cols<true>(v, col0, L + i_q0 - tile_base, rs0);
            else row_sum_cols<false>(v, col0, 0, rs0);
          } else {
            if (masked) row_sum_cols<true>(v, col0, L + i_q1 - tile_base, rs1);
            else row_sum_cols<false>(v, col0, 0, rs1);
          }
        } else if (m == 0) {
          if (masked) row_stats_cols<true>(v, col0, L + i_q0 - tile_base, c, m_raw0, z0);
          else row_stats_cols<false>(v, col0, 0, c, m_raw0, z0);
        } else {
          if (masked) row_stats_cols<true>(v, col0, L + i_q1 - tile_base, c, m_raw1, z1);
          else row_stats_cols<false>(v, col0, 0, c, m_raw1, z1);
        }
      }
    }
    // The four groups hold the statistics of the same rows over different key columns: group 3 puts its
    // pair into shared memory, groups 2 and 1 fold theirs in, group 0 folds last and stores the chunk's
    // partials (a fixed order, so the result does not depend on timing).
    float2 s0 = kFold ? make_float2(rs0.m, rs0.z) : make_float2(m_raw0 * c, z0);
    float2 s1 = kFold ? make_float2(rs1.m, rs1.z) : make_float2(m_raw1 * c, z1);
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
      float2* pbase = a.part + ((int64_t)w.chunk * a.n_kv_heads + kvh) * a.rows_pad + w.qgrp * a.rows_g;
      if (r < w.rows) pbase[r] = s0;
      if (128 + r < w.rows) pbase[128 + r] = s1;
    }
  }
  cta_epilogue(tmem_base);
}

}  // namespace qg
}  // namespace dapq
