// Importance scoring on the 5th-generation tensor cores (Section 4.2, Eq. 4):
//   S(j) = sum_i Attention(q_i, k_j),  Attention = softmax(q K^T / sqrt(d_k)),
// summed over the G query heads of a GQA group, for bf16 caches.  This is the scorer the fused
// eviction path uses; score_umma.cu holds the older form with a two-part bf16 query operand.
//
// The G*N pseudo queries of one KV head form a dense [G*N x d] block that is scored against
// every key of that head: G*N flop per byte of K, far above the HBM ridge, so the work belongs
// on tcgen05.mma with the accumulators in tensor memory.  One exponential is owed per (query,
// key) pair and per sweep, which makes the MUFU / FMA pipes the co-limiter.
//
// Two sweeps (column sums of a row-normalised matrix need every row's normaliser first):
//   sweep 1 (score_qg_sweep1.cuh)  queries on tensor-memory lanes, 192 keys per MMA: per-chunk
//             running max / sum of exp of every pseudo query;
//   sweep 2 (score_qg_sweep2.cuh)  keys on lanes, up to 256 query columns per MMA: merges the
//             partials into each query's log-sum-exp, then sums exp2(s - lse_i) per key.
//
// Precision of the query operand.  The keys are bf16 in memory and exact; a rotated query rounded
// to bf16 (8 significant bits) puts per-token scores of caches with outlier channels at the edge
// of the 2e-3 tolerance, and a second MMA pass with the rounding residual doubles the tensor work.
// Here the queries are rounded to fp16 instead (11 significant bits, 8 x finer) and the MMAs run
// fp16 x fp16: four warps rewrite every K tile from bf16 to fp16 in place in shared memory between
// its TMA arrival and its MMAs.  That conversion is exact for key magnitudes 2^-14 .. 65504 (smaller
// values round to multiples of 2^-24, larger ones saturate: caches with such keys belong on the
// two-part bf16 path, DAPQ_FLAG_Q_LO_SWEEP1 | DAPQ_FLAG_Q_LO_SWEEP2).  A caller's own bf16 queries
// (dapq_score) are exact in bf16 already: the same kernels then run bf16 x bf16 with no conversion.
//
// Work decomposition.  CTA = (chunk of K tiles, query group, KV head), one CTA per SM.  A KV head
// with more than 256 query rows is cut into equal groups (of up to 256 rows in sweep 1, up to 512 in sweep 2,
// where a CTA runs two jobs per K tile); the CTAs of one chunk sit side by side in
// the grid, run at the same time and share their K tiles through L2, so K crosses DRAM once per
// sweep whatever G*N is.  Each CTA keeps its group resident in shared memory beside a ring of K
// stages.  23 warps: warp 0 issues the TMA loads, warp 1 the MMAs (and owns tensor memory), warps
// 2-5 convert K tiles, warps 6-21 are four epilogue groups (4 warps = 128 TMEM lanes each) that
// split the columns of every accumulator, and in sweep 2 warp 22 sums the groups' partial scores.
// Every mbarrier wait is bounded: after ~1 s (or the context's own limit) the CTA raises the
// timeout status, sees its copies and MMAs in flight complete, and returns normally.
#include "score_qg_sweep1.cuh"
#include "score_qg_sweep2.cuh"

namespace dapq {
namespace {

using namespace qg;

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

// Sum of the query groups' score slots, in slot order (one thread per four scores; n4 = count / 4).
__global__ void __launch_bounds__(256)
score_slots_sum_kernel(const float4* __restrict__ slots, int n_slots, int64_t slot_stride4, float4* __restrict__ scores,
                       int64_t n4) {
  pdl_wait();
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= n4) return;
  float4 v = slots[i];
  for (int s = 1; s < n_slots; ++s) {
    const float4 u = slots[s * slot_stride4 + i];
    v.x += u.x; v.y += u.y; v.z += u.z; v.w += u.w;
  }
  scores[i] = v;
}
// The same one score per thread (arrays whose length or address is no multiple of 16 bytes).
__global__ void __launch_bounds__(256)
score_slots_sum1_kernel(const float* __restrict__ slots, int n_slots, int64_t slot_stride, float* __restrict__ scores,
                        int64_t count) {
  pdl_wait();
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= count) return;
  float v = slots[i];
  for (int s = 1; s < n_slots; ++s) v += slots[s * slot_stride + i];
  scores[i] = v;
}

}  // namespace

// 16-bit tensor [.., rows, 128] with boxes of 64 channels x box_rows rows, 128-byte swizzle.
bool encode_tile_map(CUtensorMap* map, const void* base, bool f16, int rank, const uint64_t* dims,
                     const uint64_t* strides_bytes, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t gdim[3], gstride[2];
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1}, estr[3] = {1, 1, 1};
  for (int i = 0; i < rank; ++i) gdim[i] = dims[i];
  for (int i = 0; i < rank - 1; ++i) gstride[i] = strides_bytes[i];
  return fn(map, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank,
            const_cast<void*>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Cut every sequence's keys (prompt, plus the synthetic rows if asked) into chunks of whole tiles;
// ctas_per_chunk CTAs work on every chunk (KV heads x query groups).  cta_cost: what a CTA spends besides
// its tiles (set-up, first loads, drain), in units of one tile's work.
bool plan_chunks(const SeqTable& t, int extra_keys, int tile_keys, int ctas_per_chunk, int n_sm, ChunkTable* ct,
                 double cta_cost) {
  int max_tiles = 0;
  for (int b = 0; b < t.batch; ++b) {
    const int tiles = (t.prompt_len[b] + extra_keys + tile_keys - 1) / tile_keys;
    max_tiles = tiles > max_tiles ? tiles : max_tiles;
  }
  // cost of a candidate = waves of CTAs x (tiles per CTA + fixed per-CTA work, in tile units)
  int best_c = 0;
  double best_cost = 0.0;
  for (int c = 1; c <= max_tiles; ++c) {
    int64_t n = 0;
    for (int b = 0; b < t.batch; ++b) {
      const int tiles = (t.prompt_len[b] + extra_keys + tile_keys - 1) / tile_keys;
      n += (tiles + c - 1) / c;
    }
    if (n > t.batch + kUmmaMaxChunks) continue;
    const int64_t waves = (n * ctas_per_chunk + n_sm - 1) / n_sm;
    const double cost = (double)waves * (c + cta_cost);
    if (best_c == 0 || cost < best_cost) { best_c = c; best_cost = cost; }
  }
  if (best_c == 0) return false;
  ct->chunk_tiles = best_c;
  int32_t n = 0;
  for (int b = 0; b < t.batch; ++b) {
    const int tiles = (t.prompt_len[b] + extra_keys + tile_keys - 1) / tile_keys;
    ct->cu_chunk[b] = n;
    n += (tiles + best_c - 1) / best_c;
  }
  ct->cu_chunk[t.batch] = n;
  ct->n_chunks = n;
  return true;
}

int qg_groups(const Dims& dm) { return (dm.group * dm.n_pseudo + kGroupRows - 1) / kGroupRows; }

bool qg_plan(const void* q, int q_is_f16, const CacheDev& cv, const SeqTable& t, const Dims& dm, int n_sm, QgPlan* plan) {
  const int rows_total = dm.group * dm.n_pseudo;
  plan->n_qgroups = qg_groups(dm);
  plan->rows_g = (((rows_total + plan->n_qgroups - 1) / plan->n_qgroups) + 15) & ~15;
  plan->q_is_f16 = q_is_f16;
  const int q_bytes = ((plan->rows_g + 127) / 128) * 2 * 128 * 128;
  const int s1 = (kRingEnd - (q_is_f16 ? kRefSlabBytes : 0) - q_bytes) / TileGeo<kTile1>::kStage;   // (the reference operand sits at the end)
  plan->n_stages1 = s1 < kMaxStages ? s1 : kMaxStages;
  // Sweep 2 keeps up to 512 query rows per CTA when a KV head has more than 256 (two jobs per K tile): half as
  // many CTAs fetch and convert every tile, and half as many score slots are written.
  plan->wide2 = rows_total > kGroupRows ? 1 : 0;
  plan->n_qgroups2 = plan->wide2 ? (rows_total + kWideRows - 1) / kWideRows : plan->n_qgroups;
  plan->rows_g2 = plan->wide2 ? (((rows_total + plan->n_qgroups2 - 1) / plan->n_qgroups2) + 15) & ~15 : plan->rows_g;
  const int q_bytes2 = ((plan->rows_g2 + 127) / 128) * 2 * 128 * 128;
  const int ring2 = plan->wide2 ? SmemT<true>::ring_end - (q_is_f16 ? SmemT<true>::slab_bytes : 0)
                                : kRingEnd - (q_is_f16 ? kSlabBytes : 0);                          // (the -lse operands sit at the end)
  const int s2 = (ring2 - q_bytes2) / TileGeo<kTile2>::kStage;
  plan->n_stages2 = s2 < kMaxStages ? s2 : kMaxStages;
  if (plan->n_stages1 < 2 || plan->n_stages2 < 2) return false;
  // (a sweep-2 tile is one job of about a microsecond, a sweep-1 tile two: a CTA's set-up of several
  // microseconds weighs more tiles in sweep 2, where ragged batches would otherwise be cut into waves of short CTAs)
  if (!plan_chunks(t, dm.n_pseudo, kTile1, dm.n_kv_heads * plan->n_qgroups, n_sm, &plan->ct1, 3.0)) return false;
  if (!plan_chunks(t, 0, kTile2, dm.n_kv_heads * plan->n_qgroups2, n_sm, &plan->ct2, plan->wide2 ? 3.0 : 6.0)) return false;
  // ---- tensor maps: K as [d, rows, H_kv] (one map per sweep: the boxes differ), the query operand as [d, rows]
  const uint64_t rows_k = (uint64_t)t.cu_rows[t.batch];
  const uint64_t kd[3] = {(uint64_t)kHeadDim, rows_k, (uint64_t)dm.n_kv_heads};
  uint64_t ks[2] = {(uint64_t)cv.k_row_stride * 2, (uint64_t)cv.k_head_stride * 2};
  if (dm.n_kv_heads == 1 && ks[1] == 0) ks[1] = ks[0] * rows_k;
  const uint64_t q_rows = (uint64_t)t.batch * dm.n_q_heads * dm.n_pseudo;
  const uint64_t qd[2] = {(uint64_t)kHeadDim, q_rows};
  const uint64_t qs[1] = {(uint64_t)kHeadDim * 2};
  if (ks[1] == 0 || ks[1] % 16) return false;
  return encode_tile_map(&plan->tm_k1, cv.k, false, 3, kd, ks, kTile1) && encode_tile_map(&plan->tm_k2, cv.k, false, 3, kd, ks, kTile2) &&
         encode_tile_map(&plan->tm_q, q, q_is_f16 != 0, 2, qd, qs, 128);
}

cudaError_t launch_score_qg(const QgPlan& plan, const SeqTable& t, const Dims& dm, const float* lse_in, float2* part,
                            float* slots, float* scores, int64_t score_stride, float* lse_out, const float* ref, int* status,
                            long long wait_limit, bool after_own_kernel, cudaStream_t s, LaunchLog* log) {
  Args a;
  a.n_pseudo = dm.n_pseudo;
  a.group = dm.group;
  a.n_q_heads = dm.n_q_heads;
  a.n_kv_heads = dm.n_kv_heads;
  a.rows_total = dm.group * dm.n_pseudo;
  a.n_qgroups = plan.n_qgroups;
  a.rows_g = plan.rows_g;
  a.rows_pad = (a.rows_total + 255) / 256 * 256;
  a.scale_log2e = plan.q_is_f16 ? 1.f : dm.scale_log2e;        // the library's own fp16 queries are stored times scale * log2(e)
  a.wait_limit = wait_limit > 0 ? wait_limit : kWaitLimit;
  a.part = part;
  a.ref = ref;
  a.lse_in = lse_in;
  a.lse_out = lse_out;
  a.score_stride = score_stride;
  a.slot_stride = (int64_t)dm.n_kv_heads * score_stride;
  a.scores = plan.n_qgroups2 > 1 ? slots : scores;
  a.status = status;

  auto run = [&](auto sweep1, auto sweep2, int smem2) -> cudaError_t {
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(sweep1, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(sweep2, cudaFuncAttributeMaxDynamicSharedMemorySize, smem2)) != cudaSuccess) return e;
    if (lse_in == nullptr) {
      a.n_stages = plan.n_stages1;
      a.early_loads = after_own_kernel ? 1 : 0;
      log->begin(kKindSweep1, s);
      e = launch_pdl(sweep1, dim3(plan.ct1.n_chunks * plan.n_qgroups, dm.n_kv_heads), dim3(kThreads1), kSmemBytes, s, 1,
                     plan.tm_k1, plan.tm_q, t, plan.ct1, a);
      log->end(s);
      if (e != cudaSuccess) return e;
    }
    a.n_qgroups = plan.n_qgroups2;                                       // sweep 2's own cut of the query rows
    a.rows_g = plan.rows_g2;
    a.n_stages = plan.n_stages2;
    a.early_loads = (after_own_kernel || lse_in == nullptr) ? 1 : 0;     // (sweep 1, if it ran, waited for what came before)
    log->begin(kKindSweep2, s);
    e = launch_pdl(sweep2, dim3(plan.ct2.n_chunks * plan.n_qgroups2, dm.n_kv_heads), dim3(kThreads2), smem2, s, 1,
                   plan.tm_k2, plan.tm_q, t, plan.ct2, plan.ct1, a);
    log->end(s);
    return e;
  };
  cudaError_t e;
  if (plan.wide2)
    e = plan.q_is_f16 ? run(rowstat_kernel<true>, colsum_kernel<true, true>, SmemT<true>::total)
                      : run(rowstat_kernel<false>, colsum_kernel<false, true>, SmemT<true>::total);
  else
    e = plan.q_is_f16 ? run(rowstat_kernel<true>, colsum_kernel<true, false>, kSmemBytes)
                      : run(rowstat_kernel<false>, colsum_kernel<false, false>, kSmemBytes);
  if (e != cudaSuccess) return e;
  if (plan.n_qgroups2 > 1) {
    const int64_t count = (int64_t)dm.n_kv_heads * score_stride;
    log->begin(kKindSlotSum, s);
    if (count % 4 == 0 && a.slot_stride % 4 == 0 && ((uintptr_t)slots & 15u) == 0 && ((uintptr_t)scores & 15u) == 0)
      e = launch_pdl(score_slots_sum_kernel, dim3((unsigned)((count / 4 + 255) / 256)), dim3(256), 0, s, 1,
                     (const float4*)slots, plan.n_qgroups2, a.slot_stride / 4, (float4*)scores, count / 4);
    else
      e = launch_pdl(score_slots_sum1_kernel, dim3((unsigned)((count + 255) / 256)), dim3(256), 0, s, 1, (const float*)slots,
                     plan.n_qgroups2, a.slot_stride, scores, count);
    log->end(s);
    if (e != cudaSuccess) return e;
  }
  return cudaGetLastError();
}

}  // namespace dapq
