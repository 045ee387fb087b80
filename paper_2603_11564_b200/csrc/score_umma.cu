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
//   sweep 1 (score_sweep1.cuh)  queries on tensor-memory lanes, 192 keys per MMA: per-chunk
//             running max / sum of exp of every pseudo query;
//   sweep 2 (score_sweep2.cuh)  keys on lanes, up to 256 query columns per MMA: merges the
//             partials into each query's log-sum-exp, then sums exp2(s - lse_i) per key.
// When the G*N rows of a KV head fit one block of 128 (N = 32 with G = 4) both sweeps run in a
// compact geometry: half the shared memory for the queries, a third K stage in sweep 1, and
// four accumulators of 128 columns in sweep 2.
// The rotated queries are used as a bf16 pair (hi + lo, lo = bf16(q - hi)): two MMAs per
// k-step with the same K tile.  A single bf16 rounding of q would put the per-token scores
// of caches with outlier channels outside the 2e-3 tolerance.
//
// What shaped the kernels (measured on B200): one thread can issue a tcgen05.mma about every
// 77 cycles whatever its size, so MMAs are made wide (N = 192 / 256: 105 / 139 cycles for
// 128 x N x 16) and their descriptors cost one add each; a commit -> wait -> release -> issue
// hand-off of an accumulator takes about 700 cycles, so a job is a whole [128 x 192 / 256]
// block of 16 MMAs, all epilogue groups split the columns of every job, and a warp gives the
// accumulator back the moment its last columns are in registers (what it still owes, the
// exponentials and the exchange of partial sums, needs no tensor memory).  With that, sweep 2
// runs at the pace of its MMAs; sweep 1 at the pace of its epilogue (maximum, rescaling and
// exponentials of 16 columns take a warp ~600 cycles with all sixteen at work).
//
// CTA = (chunk of K tiles, KV head); 18 warps: warp 0 issues the TMA loads (query group, K
// ring), warp 1 issues the MMAs and owns tensor memory, warps 2-17 are four epilogue groups
// (4 warps = 128 TMEM lanes each) that split the columns of every accumulator.  Every
// mbarrier wait is bounded: after ~1 s the CTA raises the timeout status, drains and returns
// normally.
#include "score_sweep1.cuh"
#include "score_sweep2.cuh"

namespace dapq {
namespace {

using namespace umma;

}  // namespace

int64_t umma_part_elems(int max_batch, int n_q_heads, int n_kv_heads, int n_pseudo) {
  const int rows_total = n_q_heads / n_kv_heads * n_pseudo;
  const int rows_pad = (rows_total + 255) / 256 * 256;          // (the compact geometry pads to 128: never more)
  return (int64_t)(max_batch + kUmmaMaxChunks) * n_kv_heads * rows_pad;
}

bool umma_plan(const void* q_hi, int has_lo, int64_t lo_row_offset, const CacheDev& cv, const SeqTable& t,
               const Dims& dm, int n_sm, UmmaPlan* plan) {
  if (!plan_chunks(t, dm.n_pseudo, kTile1, dm.n_kv_heads, n_sm, &plan->ct1)) return false;
  if (!plan_chunks(t, 0, kTile2, dm.n_kv_heads, n_sm, &plan->ct2)) return false;
  plan->has_lo = has_lo;
  plan->lo_sweep1 = plan->lo_sweep2 = has_lo;
  plan->lo_row_offset = lo_row_offset;
  // ---- tensor maps: K as [d, rows, H_kv] (one map per sweep: the boxes differ), the query operand as [d, rows]
  const uint64_t rows_k = (uint64_t)t.cu_rows[t.batch];
  const uint64_t kd[3] = {(uint64_t)kHeadDim, rows_k, (uint64_t)dm.n_kv_heads};
  uint64_t ks[2] = {(uint64_t)cv.k_row_stride * 2, (uint64_t)cv.k_head_stride * 2};
  if (dm.n_kv_heads == 1 && ks[1] == 0) ks[1] = ks[0] * rows_k;
  const uint64_t q_rows = (uint64_t)t.batch * dm.n_q_heads * dm.n_pseudo;
  const uint64_t qd[2] = {(uint64_t)kHeadDim, has_lo ? (uint64_t)lo_row_offset + q_rows : q_rows};
  const uint64_t qs[1] = {(uint64_t)kHeadDim * 2};
  if (ks[1] == 0 || ks[1] % 16) return false;
  return encode_tile_map(&plan->tm_k1, cv.k, false, 3, kd, ks, kTile1) && encode_tile_map(&plan->tm_k2, cv.k, false, 3, kd, ks, kTile2) &&
         encode_tile_map(&plan->tm_q, q_hi, false, 2, qd, qs, 128);
}

cudaError_t launch_score_umma(const UmmaPlan& plan, const SeqTable& t, const Dims& dm, const float* lse_in,
                              float2* part, float* scores, int64_t score_stride, float* lse_out,
                              int* status, long long wait_limit, cudaStream_t s, LaunchLog* log) {
  UmmaArgs a;
  a.n_pseudo = dm.n_pseudo;
  a.group = dm.group;
  a.n_q_heads = dm.n_q_heads;
  a.n_kv_heads = dm.n_kv_heads;
  a.rows_total = dm.group * dm.n_pseudo;
  const bool compact = a.rows_total <= Geo<true>::kRows;
  const int group_rows = compact ? Geo<true>::kRows : Geo<false>::kRows;
  a.n_qgroups = (a.rows_total + group_rows - 1) / group_rows;
  a.rows_pad = a.n_qgroups * group_rows;
  a.has_lo = plan.has_lo;
  a.lo_row_offset = (int32_t)plan.lo_row_offset;
  a.scale_log2e = dm.scale_log2e;
  a.wait_limit = wait_limit > 0 ? wait_limit : ptx::kWaitLimit;
  a.part = part;
  a.lse_in = lse_in;
  a.lse_out = lse_out;
  a.scores = scores;
  a.score_stride = score_stride;
  a.status = status;

  auto run = [&](auto sweep1, auto sweep2) -> cudaError_t {
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(sweep1, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(sweep2, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes)) != cudaSuccess) return e;
    if (lse_in == nullptr) {
      a.has_lo = plan.lo_sweep1;
      log->begin(kKindSweep1, s);
      e = launch_pdl(sweep1, dim3(plan.ct1.n_chunks, dm.n_kv_heads), dim3(kThreads), kSmemBytes, s, 1, plan.tm_k1, plan.tm_q, t,
                     plan.ct1, a);
      log->end(s);
      if (e != cudaSuccess) return e;
    }
    a.has_lo = plan.lo_sweep2;
    log->begin(kKindSweep2, s);
    e = launch_pdl(sweep2, dim3(plan.ct2.n_chunks, dm.n_kv_heads), dim3(kThreads), kSmemBytes, s, 1, plan.tm_k2, plan.tm_q, t,
                   plan.ct2, plan.ct1, a);
    log->end(s);
    return e;
  };
  const cudaError_t e = !compact          ? run(score_sweep1_kernel<false>, score_sweep2_kernel<false, false>)
                        : plan.lo_sweep2  ? run(score_sweep1_kernel<true>, score_sweep2_kernel<true, true>)
                                          : run(score_sweep1_kernel<true>, score_sweep2_kernel<true, false>);
  if (e != cudaSuccess) return e;
  return cudaGetLastError();
}

}  // namespace dapq
