// Sweep 2 of the tensor-core scorer (Section 4.2, Eq. 4): S(j) = sum_i exp(s_ij - lse_i),
// summed over the N pseudo queries and the G query heads of the KV head's group.
//
//   D[key, query] = K_tile Q_grp^T, keys on tensor-memory lanes, up to 256 query columns.
// CTA = (chunk of K tiles, query group, KV head): a KV head with more than 512 query rows is cut into
// groups of equal size (a CTA keeps up to 512 rows resident and then runs two jobs per K tile), each scored by a CTA of its own against the same K chunk (the CTAs of a chunk
// are neighbours in the grid, run at the same time and find each other's K tiles in L2, so K crosses
// DRAM once); the groups' scores go to separate slots that a small kernel sums in fixed order.
// A job is one [128 keys x <= 256 queries] accumulator (two fit; four of 128 columns for small groups).
// All four epilogue groups work on every job, a quarter of the query columns each, and give the
// accumulator back as soon as their columns are in registers.  No epilogue warp waits for another one:
// a warp posts its 32 partial sums into a ring of kExchDepth slots in shared memory and goes on to the
// next job; one more warp sums the four groups' entries (fixed order) and stores the keys' scores, one
// coalesced fp32 per lane.  Before the first job the epilogue threads merge the per-chunk partials of
// sweep 1 into the base-2 log-sum-exp of the resident query rows.
#pragma once
#include "score_qg_common.cuh"

namespace dapq {
namespace qg {

// 16 accumulator columns of one key row: sum of 2^(s c - lse) over the columns, as two packed pairs.
// kFull: all 16 columns exist (no per-column test).  kFold: the accumulator already holds s c - lse (the
// queries were scaled before the MMAs and -lse was added by the job's last k-step).
template <bool kFull, bool kFold>
__device__ __forceinline__ void colsum_piece(const uint32_t* v, const float* lse16, int valid, float c, float2& acc, float2& acc1) {
  if (kFull) {
    const float2 c2 = make_float2(c, c);
#pragma unroll
    for (int e = 0; e < 16; e += 4) {
      float2 x0, x1;
      if (kFold) {
        x0 = make_float2(__uint_as_float(v[e]), __uint_as_float(v[e + 1]));
        x1 = make_float2(__uint_as_float(v[e + 2]), __uint_as_float(v[e + 3]));
      } else {
        const float4 l4 = *reinterpret_cast<const float4*>(lse16 + e);
        x0 = __ffma2_rn(make_float2(__uint_as_float(v[e]), __uint_as_float(v[e + 1])), c2, make_float2(l4.x, l4.y));
        x1 = __ffma2_rn(make_float2(__uint_as_float(v[e + 2]), __uint_as_float(v[e + 3])), c2, make_float2(l4.z, l4.w));
      }
      acc = __fadd2_rn(acc, ((kPolyPairMask >> (e / 2)) & 1u) ? ex2_pair_poly(x0) : ex2_pair_mufu(x0));
      acc1 = __fadd2_rn(acc1, ((kPolyPairMask >> (e / 2 + 1)) & 1u) ? ex2_pair_poly(x1) : ex2_pair_mufu(x1));
    }
  } else {
#pragma unroll
    for (int e = 0; e < 16; ++e)
      if (e < valid) acc.x += kFold ? ex2(__uint_as_float(v[e])) : ex2(fmaf(__uint_as_float(v[e]), c, lse16[e]));
  }
}

// This warp's pieces [p0, p0 + np) of one accumulator (np <= 4), two at a time; `release` gives the
// accumulator back once the last piece is in registers.  kFull: every column of these pieces exists.
template <bool kFull, bool kFold, class Release>
__device__ __forceinline__ float colsum_job(uint32_t taddr, const float* lse_s, int p0, int np, int rows, float c, Release release) {
  float2 acc = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
  if (np == 0) release();
#pragma unroll
  for (int k = 0; k < 4; k += 2) {
    if (k < np) {
      const int ch = p0 + k;
      const int valid = rows - ch * 16;                         // >= 16 except in the last piece
      if (k + 1 < np) {
        uint32_t v[32];
        tmem_ld16(taddr + ch * 16, v);
        tmem_ld16(taddr + ch * 16 + 16, v + 16);
        tmem_ld_wait_for(v);
        if (k + 2 >= np) release();
        colsum_piece<kFull, kFold>(v, lse_s + ch * 16, valid, c, acc, acc1);
        colsum_piece<kFull, kFold>(v + 16, lse_s + ch * 16 + 16, valid - 16, c, acc, acc1);
      } else {
        uint32_t v[16];
        tmem_ld16(taddr + ch * 16, v);
        tmem_ld_wait_for16(v);
        release();
        colsum_piece<kFull, kFold>(v, lse_s + ch * 16, valid, c, acc, acc1);
      }
    }
  }
  return (acc.x + acc.y) + (acc1.x + acc1.y);
}

// kWide: the CTA keeps up to 512 query rows resident and runs two jobs per K tile (query columns 0..255 and
// 256..); a thread adds its two jobs' sums before it posts them, so a tile is fetched, converted and stored once
// for twice the queries.
template <bool kConvert, bool kWide>
__global__ void __launch_bounds__(kThreads2, 1)
colsum_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_q,
              const __grid_constant__ SeqTable t, const __grid_constant__ ChunkTable ct,
              const __grid_constant__ ChunkTable ct1, const Args a) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  if (sbase & 1023u) {                                          // (uniform over the CTA: nothing has been set up yet)
    if (threadIdx.x == 0) atomicOr(a.status, kStatusSmemAlign);
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  using T = TileGeo<kTile2>;
  constexpr bool kFold = kConvert;                              // the library's own fp16 queries arrive scaled: -lse rides on the MMAs
  const int kvh = blockIdx.y;
  const Work w = cta_work(t, ct, a, kTile2, false);
  const int nt = w.nt, L = w.L, b = w.b;
  if (nt <= 0) return;
  using Smem = SmemT<kWide>;
  const Bars bars{sbase + Smem::bars};
  const Waiter wt{reinterpret_cast<volatile int*>(smem + Smem::abort_flag), a.status, a.wait_limit};
  float* lse_s = reinterpret_cast<float*>(smem + Smem::lse);    // [rows] minus the base-2 lse of the resident query rows
  float* aux = reinterpret_cast<float*>(smem + Smem::aux);      // [rows] scratch of the lse merge
  float* exch = reinterpret_cast<float*>(smem + Smem::exch);    // [kExchDepth][4][128] partial sums on their way to the summing warp
  // The epilogue threads ask for sweep 1's partials of their query row first of all, before the CTA's copies of
  // queries and keys crowd the memory system (two threads per row: thread (eg, r) takes row (eg & 1) * 128 + r and
  // the chunks of parity eg >> 1; up to 16 partials per thread at once.  kWide: one thread per row, every chunk).
  const bool is_epi = warp >= kFirstEpiWarp && warp < kFirstEpiWarp + 4 * kEpiGroups;
  const int m_eg = (warp - kFirstEpiWarp) >> 2, m_row = (kWide ? m_eg : (m_eg & 1)) * 128 + (warp & 3) * 32 + lane;
  constexpr int m_cs = kWide ? 1 : 2;                           // chunk stride of a thread
  const int m_c0 = kWide ? 0 : (m_eg >> 1);                     // its first chunk
  const bool m_live = is_epi && m_row < w.rows && !a.lse_in;
  const int m_nc = ct1.cu_chunk[b + 1] - ct1.cu_chunk[b];
  const int64_t m_step = (int64_t)a.n_kv_heads * a.rows_pad;
  const float2* m_p = a.part + ((int64_t)ct1.cu_chunk[b] * a.n_kv_heads + kvh) * a.rows_pad + w.qgrp * a.rows_g + m_row;
  float2 m_q[16];
  if (m_live) {
    pdl_wait();                                                 // (sweep 1 wrote them)
#pragma unroll
    for (int u = 0; u < 16; ++u)
      m_q[u] = m_c0 + m_cs * u < m_nc ? __ldg(m_p + (m_c0 + m_cs * u) * m_step) : make_float2(-CUDART_INF_F, 0.f);
  }
  // (behind this library's own sweep 1 or rotation kernel, keys and queries were complete before that kernel
  // got past its wait: both go out at once)
  const uint32_t tmem_base = cta_prologue<Smem>(smem, sbase, bars, [&] {
    if (a.early_loads) tma_first<kTile2, true>(&tm_k, &tm_q, w, a, sbase, bars, kvh);
  });
  // UMMA N: only the query columns that exist; job 1 (kWide) holds the rows from 256 on
  const int ncols = (min(w.rows, kGroupRows) + 15) & ~15, ncols1 = kWide ? ((max(w.rows - kGroupRows, 0) + 15) & ~15) : 0;
  const int n_jobs = ncols1 > 0 ? 2 : 1;                        // jobs per K tile
  const int acc_cols = ncols > 128 ? 256 : 128, n_acc = kTmemCols / acc_cols;
  const uint32_t q_half = (uint32_t)w.mb * 128u * 128u;         // bytes of one 64-channel half of the query group
  const int S = a.n_stages;

  if (warp == 0) {
    if (lane == 0) {
      if (!a.early_loads) tma_first<kTile2, true>(&tm_k, &tm_q, w, a, sbase, bars, kvh);
      tma_producer<kTile2, false, true>(&tm_k, &tm_q, w, a, sbase, bars, kvh, wt);
    }
  } else if (warp == 1) {
    // ============================================================================= MMA issuer
    if (lane == 0) {
      bool ok = wt.wait(bars.q_full(), 0);
      if (ok && kFold) ok = wt.wait(bars.lse_ready(), 0);
      const uint32_t idesc = kConvert ? umma_idesc_f16(128, ncols) : umma_idesc(128, ncols);
      const uint32_t idesc1 = ncols1 ? (kConvert ? umma_idesc_f16(128, ncols1) : umma_idesc(128, ncols1)) : 0u;
      const uint64_t qd = umma_desc(sbase);
      const uint64_t ones_d = umma_desc_rows32(sbase + Smem::ones_slab), lse_d = umma_desc_rows32(sbase + Smem::lse_slab);
      const uint32_t ring = sbase + 2 * q_half;
      Ring rs(S), ra(n_acc);
      for (int ti = 0; ti < nt && ok; ++ti, rs.next()) {
        const int s = rs.i;
        ok = wt.wait(kConvert ? bars.k_conv(s) : bars.k_full(s), rs.phase);
        const uint64_t kd = umma_desc(ring + s * T::kStage);
        for (int jb = 0; jb < n_jobs && ok; ++jb, ra.next()) {
          const int buf = ra.i;
          if (ra.wrapped) ok = wt.wait(bars.acc_empty(buf), ra.phase ^ 1u);
          if (!ok) break;
          tc_fence_after();
          const uint32_t d = tmem_base + buf * acc_cols;
          const uint64_t qj = desc_advance(qd, jb * 2 * 128 * 128);          // query rows 256 jb ..: blocks 2 jb, 2 jb + 1
          const uint32_t id = jb ? idesc1 : idesc;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const int half = ks >> 2, kk = ks & 3;
            umma_ss(d, desc_advance(kd, half * T::kHalf + kk * 32), desc_advance(qj, half * q_half + kk * 32), id, ks ? 1u : 0u);
          }
          // D[key, i] += 1 * (-lse_i) (an fp16 pair against two ones)
          if (kFold) umma_ss(d, ones_d, desc_advance(lse_d, jb * kGroupRows * 32), id, 1u);
          tc_commit(bars.acc_full(buf));
        }
        if (!ok) break;
        tc_commit(bars.k_empty(s));                             // the K stage is free once these MMAs retire
      }
      mma_drain(bars);
    }
  } else if (warp < kFirstEpiWarp) {
    if (kConvert) convert_tiles<kTile2>(w, a, sbase, bars, warp - 2, wt);
  } else if (warp < kFirstEpiWarp + 4 * kEpiGroups) {
    // ============================================================================== epilogue
    const int eg = (warp - kFirstEpiWarp) >> 2;                 // epilogue group 0 .. 3
    const int quad = warp & 3;                                  // TMEM lane quadrant of this warp
    const int r = quad * 32 + lane;                             // accumulator row (key) of this thread
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float c = a.scale_log2e;
    // ---- base-2 log-sum-exp of the group's rows.  Two threads per row: thread (eg, r) merges the per-chunk
    // partials of row (eg & 1) * 128 + r over the chunks of parity eg >> 1, all of its loads in flight at
    // once; the odd half then crosses through shared memory and the even half finishes (fixed order).
    {
      const int row = m_row, grow = w.qgrp * a.rows_g + row;
      const bool live = row < w.rows;
      float mx = -CUDART_INF_F, z = 0.f;
      if (m_live) {
        for (int c0 = m_c0; c0 < m_nc; c0 += 16 * m_cs) {
          if (c0 > m_c0) {                                      // (more chunks than one batch of 16 per thread)
#pragma unroll
            for (int u = 0; u < 16; ++u)
              m_q[u] = c0 + m_cs * u < m_nc ? __ldg(m_p + (c0 + m_cs * u) * m_step) : make_float2(-CUDART_INF_F, 0.f);
          }
          float m16 = m_q[0].x;
#pragma unroll
          for (int u = 1; u < 16; ++u) m16 = fmaxf(m16, m_q[u].x);
          if (m16 > mx) {
            z *= exp2f(mx - m16);                               // exp2f(-inf) = 0 on the first round
            mx = m16;
          }
          if (mx > -CUDART_INF_F) {
#pragma unroll
            for (int u = 0; u < 16; ++u) z += m_q[u].y * exp2f(m_q[u].x - mx);
          }
        }
      }
      if (!kWide && eg >= 2) {
        aux[row] = mx;
        lse_s[row] = z;                                         // (the odd half's sums, until the even half has read them)
      }
      epilogue_sync();
      if (kWide || eg < 2) {
        float l2 = 0.f;
        if (live) {
          if (a.lse_in) {
            l2 = a.lse_in[w.qrow_base + grow] * 1.4426950408889634f;
          } else if (kWide) {
            l2 = mx + log2f(z);
          } else {
            const float mo = aux[row], zo = lse_s[row];
            const float m = fmaxf(mx, mo);
            l2 = m + log2f(z * exp2f(mx - m) + zo * exp2f(mo - m));
          }
          if (a.lse_out && w.chunk == ct.cu_chunk[b]) a.lse_out[w.qrow_base + grow] = l2 * 0.6931471805599453f;
        }
        lse_s[row] = -l2;                                       // negated: the epilogue adds it
        if (kFold) {
          // row `row` of the [256 x 16] operand: (-lse) as an fp16 pair in channels 0 and 1, zeros elsewhere.
          // The ones operand carries its two ones in BOTH 16-byte halves of every row, so whichever way the
          // 32-byte swizzle orders the halves of a row, the k-step adds exactly hi + lo.
          const __half hi = __float2half_rn(-l2);
          const __half lo = __float2half_rn(live ? -l2 - __half2float(hi) : 0.f);
          const uint32_t pair = (uint32_t)__half_as_ushort(hi) | ((uint32_t)__half_as_ushort(lo) << 16);
          const uint32_t dst = sbase + Smem::lse_slab + (row >> 3) * 256 + (row & 7) * 32;
          sts128(dst, make_uint4(live ? pair : 0u, 0u, 0u, 0u));
          sts128(dst + 16, make_uint4(0u, 0u, 0u, 0u));
        }
      }
      if (kFold) {
        const int tid_e = (warp - kFirstEpiWarp) * 32 + lane;   // 0 .. 511: the ones operand, 256 pieces of 16 bytes
        if (tid_e < kOnesSlabBytes / 16) sts128(sbase + Smem::ones_slab + tid_e * 16, make_uint4(0x3c003c00u, 0u, 0u, 0u));
        fence_proxy_async();                                    // the MMAs read both operands through the async proxy
      }
      epilogue_sync();
      if (warp == kFirstEpiWarp && lane == 0) mbar_arrive(bars.lse_ready());    // (the MMA issuer and the TMA producer wait for it)
    }
    // Pieces of a job (16 query columns): group g takes pieces [g nch / 4, (g + 1) nch / 4), at most four
    const int nch = ncols >> 4, nch1 = ncols1 >> 4;
    const int p0 = (eg * nch) / kEpiGroups, np = ((eg + 1) * nch) / kEpiGroups - p0;
    const int p1 = (eg * nch1) / kEpiGroups, np1 = ((eg + 1) * nch1) / kEpiGroups - p1;
    const bool full = (p0 + np) * 16 <= min(w.rows, kGroupRows);    // no column of this warp's pieces lies beyond the group
    const bool full1 = (p1 + np1) * 16 <= w.rows - kGroupRows;
    bool ok = true;
    Ring ra(n_acc);
    for (int ti = 0; ti < nt && ok; ++ti) {
      float sum = 0.f;
      for (int jb = 0; jb < n_jobs && ok; ++jb, ra.next()) {
        const int buf = ra.i;
        ok = __all_sync(0xffffffffu, wt.wait(bars.acc_full(buf), ra.phase));
        if (!ok) break;
        tc_fence_after();
        const uint32_t taddr = lane_addr + buf * acc_cols;
        // the accumulator goes back to the MMA issuer as soon as this warp's last piece is in registers
        auto release = [&] {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bars.acc_empty(buf));
        };
        if (jb == 0)
          sum = full ? colsum_job<true, kFold>(taddr, lse_s, p0, np, min(w.rows, kGroupRows), c, release)
                     : colsum_job<false, kFold>(taddr, lse_s, p0, np, min(w.rows, kGroupRows), c, release);
        else
          sum += full1 ? colsum_job<true, kFold>(taddr, lse_s + kGroupRows, p1, np1, w.rows - kGroupRows, c, release)
                       : colsum_job<false, kFold>(taddr, lse_s + kGroupRows, p1, np1, w.rows - kGroupRows, c, release);
      }
      if (!ok) break;
      const int slot = ti % kExchDepth;
      if (ti >= kExchDepth) ok = __all_sync(0xffffffffu, wt.wait(bars.part_empty(slot), ((ti / kExchDepth) - 1) & 1));
      if (!ok) break;
      exch[(slot * kEpiGroups + eg) * 128 + r] = sum;
      __syncwarp();
      if (lane == 0) mbar_arrive(bars.part_full(slot));         // (release: the stores above are visible to the waiter)
    }
  } else {
    // ====================================================================== sum of the four groups
    float* out = a.scores + (int64_t)w.qgrp * a.slot_stride + (int64_t)kvh * a.score_stride + t.cu_prompt[b];
    for (int ti = 0; ti < nt; ++ti) {
      const int slot = ti % kExchDepth;
      if (!__all_sync(0xffffffffu, wt.wait(bars.part_full(slot), (ti / kExchDepth) & 1))) break;
      const float* e = exch + slot * kEpiGroups * 128;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int r = q * 32 + lane;
        const float v = ((e[r] + e[128 + r]) + e[256 + r]) + e[384 + r];
        const int j = (w.t0 + ti) * kTile2 + r;                 // sequence-local key position
        if (j < L) out[j] = v;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bars.part_empty(slot));
    }
  }
  cta_epilogue(tmem_base);
}

}  // namespace qg
}  // namespace dapq
