// Internal declarations shared by the translation units of libdapq (not installed).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dapq.h"

namespace dapq {

constexpr int kHeadDim = DAPQ_HEAD_DIM;      // d
constexpr int kMaxBatch = DAPQ_MAX_BATCH;
constexpr int kMaxPseudo = DAPQ_MAX_PSEUDO;
constexpr int kChunkKeys = 512;              // most prompt keys per work chunk of the CUDA-core score sweeps

// Per-call sequence geometry, passed by value to the kernels (host arrays never have to
// be copied to the device, so a call adds no copy nodes to a stream).
struct SeqTable {
  int32_t batch;
  int32_t cu_rows[kMaxBatch + 1];   // first cache row of sequence b
  int32_t cu_prompt[kMaxBatch + 1]; // first score column of sequence b
  int32_t cu_keep[kMaxBatch + 1];   // first output row of sequence b (K_b clamped to L_b)
  int32_t prompt_len[kMaxBatch];    // L_b
  int32_t pos_start[kMaxBatch];     // position of pseudo query 0
};

// How the score sweeps cut the sequences into work chunks (one CTA per chunk and KV head).
//   CUDA-core path:   chunks of chunk_tiles prompt KEYS (64 .. kChunkKeys), then one chunk with the N
//                     synthetic rows;
//   tensor-core path: chunks of chunk_tiles whole K tiles (the tile size is the sweep's).
struct ChunkTable {
  int32_t chunk_tiles;
  int32_t n_chunks;
  int32_t cu_chunk[kMaxBatch + 1];  // first chunk of sequence b
};
constexpr int kUmmaMaxChunks = 256;  // the tensor-core planner never makes more chunks than max_batch + this

struct CacheDev {
  const void* k;
  const void* v;
  int64_t k_head_stride, k_row_stride, v_head_stride, v_row_stride;  // elements
};

struct Dims {
  int32_t n_q_heads, n_kv_heads, group, n_pseudo;
  float scale_log2e;                // softmax scale * log2(e): logits are kept in base 2
  int32_t rope_interleaved = 0;     // RoPE pairs are (2c, 2c + 1) instead of (c, c + d/2)
};

// Device status word bits (set by kernels, read by dapq_poll_status).
enum : int { kStatusTimeout = 1, kStatusBadIndex = 2, kStatusSmemAlign = 4 };

// Output formats of the rotation kernel.
enum : int { kRopeOutBf16 = DAPQ_BF16, kRopeOutF32 = DAPQ_F32, kRopeOutSplitBf16 = 2, kRopeOutF16 = 3 };

__device__ __forceinline__ int find_segment(const int32_t* cu, int n, int x) {
  // largest b in [0, n) with cu[b] <= x
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (cu[mid] <= x) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// Kernel kinds, for launch accounting and the optional per-kernel event timing.
enum KernelKind : int { kKindRope = 0, kKindSweep1, kKindLseMerge, kKindSweep2, kKindTopk, kKindCompact, kKindPool,
                        kKindRecall, kKindSlotSum, kKindCount };

// Counts launches and, while profiling is on, brackets every launch with CUDA events on
// the launching stream (implemented in api.cu; events come from a host-side pool).
struct LaunchLog {
  int64_t n_launch = 0;
  bool profiling = false;
  void* impl = nullptr;
  void begin(int kind, cudaStream_t s);
  void end(cudaStream_t s);
};

// ---- programmatic dependent launch --------------------------------------------------------
// Every kernel of the eviction path is launched with programmatic stream serialization and
// waits, before its first access to global memory, until the kernel before it has completed
// and its writes are visible (pdl_wait): its launch is then prepared, and its CTAs' set-up done,
// while the predecessor still runs.  The short kernels that precede a long one (rotation,
// selection) also signal at their start that the next kernel may be scheduled (pdl_trigger); the
// sweeps do not: their successors' CTAs would only sit on the SMs the next sweep needs (measured:
// slower).  The compaction signals at its start too: in dapq_evict_layers the next layer's
// rotation, which touches nothing the compaction or the selection before it use, runs beside
// them and waits at its END, so that the kernels after it stay ordered behind the compaction.
// Both instructions are no-ops for a kernel launched the ordinary way.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Launch with programmatic stream serialization (and a cluster of cluster_x CTAs if > 1).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, int cluster_x,
                       Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  int n = 0;
  attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster_x;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- launchers (each returns the cudaError_t of its launch) -------------------------------
// q_pre has element type `dtype`; q_rot is written as `out_mode`: bf16, fp32 (unrounded, for
// the CUDA-core scorer) or a bf16 pair hi + lo with lo = bf16(q - hi) stored `lo_offset`
// elements after hi (for the tensor-core scorer).
// ref (fp16 output mode only, may be NULL): the bf16 key cache and where to write, per rotated query, its base-2
// logit against the first key of its sequence (see rope.cu).
struct RopeRef {
  const __nv_bfloat16* k;
  int64_t head_stride, row_stride;   // elements
  float* out;                        // [B, H_q, N]
  int32_t group;
};
cudaError_t launch_rope(int dtype, int out_mode, int64_t lo_offset, const void* q_pre, void* q_rot, const double* inv_freq_dev,
                        const SeqTable& t, const Dims& dm, bool late_wait, cudaStream_t s, LaunchLog* log,
                        const RopeRef* ref = nullptr);

// Generic CUDA-core scorer (any N <= 128, both dtypes).
//   part  : [n_chunks, H_q, N] float2 (running max, sum) in base-2 logits, room for max_chunks
//           chunks (at least the count at kChunkKeys keys per chunk; more lets small inputs
//           be cut finer so that they fill the n_sm SMs)
//   lse2  : [B, H_q, N] base-2 log-sum-exp
cudaError_t launch_score_fma(int dtype, int q_dtype, const void* q_rot, const CacheDev& cv, const SeqTable& t,
                             const Dims& dm, const float* lse_in, float2* part, int64_t max_chunks, int n_sm,
                             float* lse2, float* scores, int64_t score_stride, float* lse_out, float* syn_mass,
                             cudaStream_t s, LaunchLog* log);

// Makes the device code of every CUDA-core score kernel resident on the current device (no launch).
cudaError_t score_fma_preload();

// Tensor-core scorer (bf16 caches).  umma_plan encodes the TMA descriptors and cuts the work;
// it returns false when the view cannot be described to TMA (the caller then takes the
// CUDA-core path).  q_hi: [B*H_q*N, d] bf16; with has_lo the low-order parts follow
// lo_row_offset rows later in the same allocation.
struct UmmaPlan {
  CUtensorMap tm_k1, tm_k2, tm_q;   // K for sweep 1 / sweep 2 (different boxes), the query operand
  ChunkTable ct1, ct2;              // work cut of sweep 1 (192-key tiles over L_b + N) / sweep 2 (128-key tiles over L_b)
  int32_t has_lo;                   // the low-order parts exist in memory
  int32_t lo_sweep1, lo_sweep2;     // ... and which sweep adds them (a second MMA pass)
  int64_t lo_row_offset;
};
bool umma_plan(const void* q_hi, int has_lo, int64_t lo_row_offset, const CacheDev& cv, const SeqTable& t,
               const Dims& dm, int n_sm, UmmaPlan* plan);
int64_t umma_part_elems(int max_batch, int n_q_heads, int n_kv_heads, int n_pseudo);
cudaError_t launch_score_umma(const UmmaPlan& plan, const SeqTable& t, const Dims& dm, const float* lse_in,
                              float2* part, float* scores, int64_t score_stride, float* lse_out,
                              int* status, long long wait_limit, cudaStream_t s, LaunchLog* log);

// Pieces shared by the two tensor-core scorers (defined in score_qg.cu): the TMA descriptor of a
// 16-bit [.., rows, 128] tensor (boxes of 64 channels x box_rows rows, 128-byte swizzle), and the cut of
// the sequences' keys into chunks of whole tiles with ctas_per_chunk CTAs working on every chunk.
bool encode_tile_map(CUtensorMap* map, const void* base, bool f16, int rank, const uint64_t* dims,
                     const uint64_t* strides_bytes, int box_rows);
bool plan_chunks(const SeqTable& t, int extra_keys, int tile_keys, int ctas_per_chunk, int n_sm, ChunkTable* ct,
                 double cta_cost = 3.0);

// Tensor-core scorer with one query group per CTA (score_qg.cu).  q: [B*H_q*N, d], fp16 (the K tiles
// are then converted to fp16 in shared memory) or bf16.  qg_plan returns false when the view cannot be
// described to TMA.  With more than one query group per KV head the sweeps write one score slot per
// group into `slots` ([n_qgroups, H_kv, score_stride]) and a last kernel sums them into `scores`.
struct QgPlan {
  CUtensorMap tm_k1, tm_k2, tm_q;
  ChunkTable ct1, ct2;
  int32_t n_qgroups, rows_g, n_stages1, n_stages2, q_is_f16;
  int32_t n_qgroups2, rows_g2, wide2;     // sweep 2's own cut of the query rows (groups of up to 512 rows when wide2)
};
int qg_groups(const Dims& dm);
bool qg_plan(const void* q, int q_is_f16, const CacheDev& cv, const SeqTable& t, const Dims& dm, int n_sm, QgPlan* plan);
// ref: with fp16 queries, the [B, H_q, N] reference logits that the rotation kernel wrote beside them.
// after_own_kernel: the kernel before these in the stream is this library's rotation kernel (which waits for
// whatever precedes it), so the sweeps may copy the keys before their own wait for it.
cudaError_t launch_score_qg(const QgPlan& plan, const SeqTable& t, const Dims& dm, const float* lse_in, float2* part,
                            float* slots, float* scores, int64_t score_stride, float* lse_out, const float* ref, int* status,
                            long long wait_limit, bool after_own_kernel, cudaStream_t s, LaunchLog* log);

cudaError_t launch_topk(const float* scores, int64_t score_stride, int32_t* idx, int64_t idx_stride,
                        const SeqTable& t, int n_kv_heads, cudaStream_t s, LaunchLog* log);

// pooled[kvh, j] = max / mean of scores[kvh, j - kernel/2 .. j + kernel/2] within each sequence.
cudaError_t launch_pool(const float* scores, float* pooled, int64_t stride, const SeqTable& t, int n_kv_heads,
                        int kernel, int mode, cudaStream_t s, LaunchLog* log);

// recall[b, kvh] = |gold ∩ pred| / |gold| for two ascending index lists per (sequence, KV head).
cudaError_t launch_recall(const int32_t* gold, const int32_t* pred, int64_t idx_stride, const SeqTable& t,
                          int n_kv_heads, float* recall, cudaStream_t s, LaunchLog* log);

cudaError_t launch_compact(int dtype, const CacheDev& cv, const int32_t* idx, int64_t idx_stride,
                           void* k_out, void* v_out, const SeqTable& t, int n_kv_heads, int* status,
                           cudaStream_t s, LaunchLog* log);

}  // namespace dapq
