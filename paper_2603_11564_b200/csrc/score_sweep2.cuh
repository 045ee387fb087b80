// Sweep 2 of the tensor-core scorer (Section 4.2, Eq. 4): S(j) = sum_i exp(s_ij - lse_i),
// summed over the N pseudo queries and the G query heads of the KV head's group.
//
//   D[key, query] = K_tile Q_grp^T, keys on tensor-memory lanes, up to 256 query columns.
// A job is one [128 keys x 256 queries] accumulator (two fit; four of 128 columns in the compact
// geometry).  In the compact geometry with a hi + lo query operand (kWide) the 128 hi rows and the
// 128 lo rows sit side by side as the 256 columns of ONE MMA per k-step: the K tile is read from
// shared memory once instead of twice (MMAs of N = 128 with both operands in shared memory are
// bound by its bandwidth), and the epilogue adds the two halves before the exponential.  All four epilogue groups work
// on every job, a quarter of the query columns each (sixteen epilogue warps, four per scheduler,
// hide the latency of the tensor-memory loads and of the hand-offs) and gives the accumulator back
// as soon as its columns are in registers; groups 1-3 hand their partial sums to group 0 through
// shared memory, and group 0's thread (lane = key) stores the key's score: one coalesced fp32 per
// lane.  Before the first job the
// epilogue threads merge the per-chunk partials of sweep 1 into the base-2 log-sum-exp of the
// resident query rows.
#pragma once
#include "score_umma_common.cuh"

namespace dapq {
namespace umma {

template <bool kCompact, bool kWide>
__global__ void __launch_bounds__(kThreads, 1)
score_sweep2_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_q,
                    const __grid_constant__ SeqTable t, const __grid_constant__ ChunkTable ct,
                    const __grid_constant__ ChunkTable ct1, const UmmaArgs a) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  if (sbase & 1023u) {                                          // (uniform over the CTA: nothing has been set up yet)
    if (threadIdx.x == 0) atomicOr(a.status, kStatusSmemAlign);
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  using G = Geo<kCompact>;
  static_assert(kCompact || !kWide, "the side-by-side operand needs the compact geometry");
  constexpr int kStages2 = G::kStages2, kAcc = kWide ? 2 : G::kAcc2, kAccCols = kTmemCols / kAcc;
  const int chunk = blockIdx.x, kvh = blockIdx.y;
  const Work w = cta_work(t, ct, a, kTile2, false);
  const int nt = w.nt, L = w.L, b = w.b;
  if (nt <= 0) return;
  const Bars bars{sbase + Smem::bars};
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + Smem::abort_flag);
  float* lse_s = reinterpret_cast<float*>(smem + Smem::lse);    // [256] minus the base-2 lse of the resident query rows
  float* exch = reinterpret_cast<float*>(smem + Smem::exch);    // [3][128] partial sums on their way to group 0
  const uint32_t tmem_base = cta_prologue(smem, sbase, bars, kStages2, kAcc);

  if (warp == 0) {
    if (lane == 0)
      tma_producer<G, kTile2, kStages2, kStageBytes2, kHalfBytes2, kWide>(&tm_k, &tm_q, w, a, sbase, bars, kvh, abort_flag);
  } else if (warp == 1) {
    // ============================================================================= MMA issuer
    if (lane == 0) {
      int job = 0, n_done = 0;                                  // job = K tiles consumed: one job per tile
      bool ok = true;
      const uint64_t qd_hi = umma_desc(sbase + G::q_hi), qd_lo = umma_desc(sbase + G::q_lo);
      for (int qg = 0; qg < a.n_qgroups && ok; ++qg) {
        const int rows_g = min(G::kRows, a.rows_total - qg * G::kRows);
        const uint32_t idesc = umma_idesc(128, kWide ? 256 : (rows_g + 15) & ~15);   // only the query columns that exist
        ok = mbar_wait_limit(bars.q_full(), qg & 1, abort_flag, a.status, a.wait_limit);
        for (int ti = 0; ti < nt && ok; ++ti, ++job) {
          const int s = job % kStages2, buf = job % kAcc;
          ok = mbar_wait_limit(bars.k_full(s), (job / kStages2) & 1, abort_flag, a.status, a.wait_limit);
          if (ok && job >= kAcc) ok = mbar_wait_limit(bars.acc_empty(buf), ((job / kAcc) - 1) & 1, abort_flag, a.status, a.wait_limit);
          if (!ok) break;
          tc_fence_after();
          const uint64_t kd = umma_desc(sbase + G::k + s * kStageBytes2);
          const uint32_t d = tmem_base + buf * kAccCols;
          if (kWide) {
            // hi and lo rows side by side: one MMA of N = 256 per k-step, columns 0-127 = K q_hi^T, 128-255 = K q_lo^T
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const int half = ks >> 2, kk = ks & 3;
              umma_ss(d, desc_advance(kd, half * kHalfBytes2 + kk * 32), desc_advance(qd_hi, half * 2 * G::kHalfBytesQ + kk * 32),
                      idesc, ks ? 1u : 0u);
            }
          } else {
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const int half = ks >> 2, kk = ks & 3;
              umma_ss(d, desc_advance(kd, half * kHalfBytes2 + kk * 32), desc_advance(qd_hi, half * G::kHalfBytesQ + kk * 32),
                      idesc, ks ? 1u : 0u);
            }
            if (a.has_lo) {
#pragma unroll
              for (int ks = 0; ks < 8; ++ks) {
                const int half = ks >> 2, kk = ks & 3;
                umma_ss(d, desc_advance(kd, half * kHalfBytes2 + kk * 32), desc_advance(qd_lo, half * G::kHalfBytesQ + kk * 32),
                        idesc, 1u);
              }
            }
          }
          tc_commit(bars.acc_full(buf));
          tc_commit(bars.k_empty(s));                           // the K stage is free once these MMAs retire
        }
        tc_commit(bars.q_empty());
        ++n_done;
      }
      mma_drain(bars, n_done, n_done < a.n_qgroups);
    }
  } else {
    // ============================================================================== epilogue
    const int eg = (warp - 2) >> 2;                             // epilogue group 0 .. 3
    const int quad = warp & 3;                                  // TMEM lane quadrant of this warp
    const int r = quad * 32 + lane;                             // accumulator row of this thread
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float c = a.scale_log2e;
    const float2 c2 = make_float2(c, c);
    int job = 0;                                                // jobs of this CTA so far
    bool ok = true;
    // (an aborting group still walks every query group: the other groups wait for it at the barriers)
    for (int qg = 0; qg < a.n_qgroups; ++qg) {
      const int rows_g = min(G::kRows, a.rows_total - qg * G::kRows);
      // ---- base-2 log-sum-exp of the group's rows.  Two threads per row: thread (eg, r) merges the per-chunk
      // partials of row (eg & 1) * 128 + r over the chunks of parity eg >> 1, all of its loads in flight at
      // once; the odd half then crosses through shared memory and the even half finishes (fixed order).
      if (qg > 0) epilogue_sync();                              // the previous group's values are no longer read
      {
        const int row = (eg & 1) * 128 + r, grow = qg * G::kRows + row;
        const bool live = row < G::kRows && grow < a.rows_total;
        float mx = -CUDART_INF_F, z = 0.f;
        if (live && !a.lse_in) {
          const float2* p = a.part + ((int64_t)ct1.cu_chunk[b] * a.n_kv_heads + kvh) * a.rows_pad + grow;
          const int64_t step = (int64_t)a.n_kv_heads * a.rows_pad;
          const int nc = ct1.cu_chunk[b + 1] - ct1.cu_chunk[b];
          for (int c0 = eg >> 1; c0 < nc; c0 += 32) {
            float2 q[16];
#pragma unroll
            for (int u = 0; u < 16; ++u)
              q[u] = c0 + 2 * u < nc ? __ldg(p + (c0 + 2 * u) * step) : make_float2(-CUDART_INF_F, 0.f);
            float m16 = q[0].x;
#pragma unroll
            for (int u = 1; u < 16; ++u) m16 = fmaxf(m16, q[u].x);
            if (m16 > mx) {
              z *= exp2f(mx - m16);                             // exp2f(-inf) = 0 on the first round
              mx = m16;
            }
            if (mx > -CUDART_INF_F) {
#pragma unroll
              for (int u = 0; u < 16; ++u) z += q[u].y * exp2f(q[u].x - mx);
            }
          }
        }
        if (eg >= 2) {                                          // (lse_s holds the odd half's sums until the even half has read them)
          exch[row] = mx;
          lse_s[row] = z;
        }
        epilogue_sync();
        if (eg < 2) {
          float l2 = 0.f;
          if (live) {
            if (a.lse_in) {
              l2 = a.lse_in[w.qrow_base + grow] * 1.4426950408889634f;
            } else {
              const float mo = exch[row], zo = lse_s[row];
              const float m = fmaxf(mx, mo);
              l2 = m + log2f(z * exp2f(mx - m) + zo * exp2f(mo - m));
            }
            if (a.lse_out && chunk == ct.cu_chunk[b]) a.lse_out[w.qrow_base + grow] = l2 * 0.6931471805599453f;
          }
          lse_s[row] = -l2;                                       // negated: the epilogue adds it
        }
      }
      epilogue_sync();
      // Pieces of a job (32 query columns; 16 with the side-by-side operand, whose two halves are added
      // first): group g takes pieces [g nch / 4, (g + 1) nch / 4), at most two
      constexpr int kPiece = kWide ? 16 : 32;
      const int nch = (rows_g + kPiece - 1) / kPiece;
      const int p0 = (eg * nch) / kEpiGroups, np = ((eg + 1) * nch) / kEpiGroups - p0;
      for (int ti = 0; ti < nt && ok; ++ti, ++job) {
        const int buf = job % kAcc;
        ok = __all_sync(0xffffffffu, mbar_wait_limit(bars.acc_full(buf), (job / kAcc) & 1, abort_flag, a.status, a.wait_limit));
        if (!ok) break;
        tc_fence_after();
        const uint32_t taddr = lane_addr + buf * kAccCols;
        float2 acc = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
        // the accumulator goes back to the MMA issuer as soon as this warp's last piece is in registers
        auto release = [&] {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bars.acc_empty(buf));
        };
        if (np == 0) release();
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          if (k < np) {
            const int ch = p0 + k;
            const int valid = rows_g - ch * kPiece;             // >= kPiece except in the last piece
            if (kWide) {
              uint32_t vh[16], vl[16];
              tmem_ld16(taddr + ch * 16, vh);                   // K q_hi^T
              tmem_ld16(taddr + 128 + ch * 16, vl);             // K q_lo^T
              tmem_ld_wait_for16(vh);
              tmem_ld_wait_for16(vl);
              if (k == np - 1) release();
              if (valid >= 16) {
#pragma unroll
                for (int e = 0; e < 16; e += 4) {
                  const float4 l4 = *reinterpret_cast<const float4*>(lse_s + ch * 16 + e);
                  const float2 s0 = __fadd2_rn(make_float2(__uint_as_float(vh[e]), __uint_as_float(vh[e + 1])),
                                               make_float2(__uint_as_float(vl[e]), __uint_as_float(vl[e + 1])));
                  const float2 s1 = __fadd2_rn(make_float2(__uint_as_float(vh[e + 2]), __uint_as_float(vh[e + 3])),
                                               make_float2(__uint_as_float(vl[e + 2]), __uint_as_float(vl[e + 3])));
                  const float2 x0 = __ffma2_rn(s0, c2, make_float2(l4.x, l4.y));
                  const float2 x1 = __ffma2_rn(s1, c2, make_float2(l4.z, l4.w));
                  acc = __fadd2_rn(acc, ((kPolyPairMask >> (e / 2)) & 1u) ? ex2_pair_poly(x0) : ex2_pair_mufu(x0));
                  acc1 = __fadd2_rn(acc1, ((kPolyPairMask >> (e / 2 + 1)) & 1u) ? ex2_pair_poly(x1) : ex2_pair_mufu(x1));
                }
              } else {
#pragma unroll
                for (int e = 0; e < 16; ++e)
                  if (e < valid) acc.x += ex2(fmaf(__uint_as_float(vh[e]) + __uint_as_float(vl[e]), c, lse_s[ch * 16 + e]));
              }
            } else {
              uint32_t v[32];
              tmem_ld32(taddr + ch * 32, v);
              tmem_ld_wait_for(v);
              if (k == np - 1) release();
              if (valid >= 32) {
                // pairs of columns on the packed fp32 pipe: x = s * c - lse, then 2^x by MUFU or polynomial
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                  const float4 l4 = *reinterpret_cast<const float4*>(lse_s + ch * 32 + e);
                  const float2 x0 = __ffma2_rn(make_float2(__uint_as_float(v[e]), __uint_as_float(v[e + 1])), c2,
                                               make_float2(l4.x, l4.y));
                  const float2 x1 = __ffma2_rn(make_float2(__uint_as_float(v[e + 2]), __uint_as_float(v[e + 3])), c2,
                                               make_float2(l4.z, l4.w));
                  acc = __fadd2_rn(acc, ((kPolyPairMask >> (e / 2)) & 1u) ? ex2_pair_poly(x0) : ex2_pair_mufu(x0));
                  acc1 = __fadd2_rn(acc1, ((kPolyPairMask >> (e / 2 + 1)) & 1u) ? ex2_pair_poly(x1) : ex2_pair_mufu(x1));
                }
              } else {
#pragma unroll
                for (int e = 0; e < 32; ++e)
                  if (e < valid) acc.x += ex2(fmaf(__uint_as_float(v[e]), c, lse_s[ch * 32 + e]));
              }
            }
          }
        }
        float sum = (acc.x + acc.y) + (acc1.x + acc1.y);
        // Groups 1-3 hand their partial sums to group 0 through one slot of shared memory: the slot is
        // written once group 0 has read the job before (part_empty) and read once all three have
        // written (part_full).
        if (eg > 0) {
          if (job > 0) ok = __all_sync(0xffffffffu, mbar_wait_limit(bars.part_empty(), (job - 1) & 1, abort_flag, a.status, a.wait_limit));
          if (!ok) break;
          exch[(eg - 1) * 128 + r] = sum;
          __syncwarp();
          if (lane == 0) mbar_arrive(bars.part_full());         // (release: the stores above are visible to the waiter)
        } else {
          ok = __all_sync(0xffffffffu, mbar_wait_limit(bars.part_full(), job & 1, abort_flag, a.status, a.wait_limit));
          if (!ok) break;
          sum += (exch[r] + exch[128 + r]) + exch[256 + r];
          __syncwarp();
          if (lane == 0) mbar_arrive(bars.part_empty());
          const int j = (w.t0 + ti) * kTile2 + r;               // sequence-local key position
          if (j < L) {
            float* out = a.scores + (int64_t)kvh * a.score_stride + t.cu_prompt[b] + j;
            *out = (qg == 0) ? sum : *out + sum;
          }
        }
      }
    }
  }
  cta_epilogue(tmem_base);
}

}  // namespace umma
}  // namespace dapq
