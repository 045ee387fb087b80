// Pruning of the cache (Section 4.2: every key-value pair outside M_retain is discarded,
// and so is the whole synthetic segment).  A bit-exact gather of 256-byte (bf16) or
// 512-byte (fp32) rows: one thread per 16-byte piece, K and V in the same launch.
// Pure HBM traffic: rows_kept * row_bytes read + the same written, for K and for V.
#include "dapq_internal.cuh"

namespace dapq {
namespace {

constexpr int kCompactThreads = 256;

template <int kPieces>   // 16-byte pieces per row
__global__ void __launch_bounds__(kCompactThreads)
compact_kv_kernel(const CacheDev cv, int elem_bytes, const int32_t* __restrict__ idx, int64_t idx_stride,
                  uint4* __restrict__ k_out, uint4* __restrict__ v_out,
                  const __grid_constant__ SeqTable t, int* __restrict__ status) {
  pdl_trigger();                     // whatever follows may be set up (or, if it does not depend on this copy, run) beside it
  pdl_wait();
  const int kt = t.cu_keep[t.batch];
  const int64_t gid = (int64_t)blockIdx.x * kCompactThreads + threadIdx.x;
  const int r = (int)(gid / kPieces), piece = (int)(gid % kPieces);
  if (r >= kt) return;
  const int kvh = blockIdx.y;
  const bool is_v = blockIdx.z != 0;
  const int b = find_segment(t.cu_keep, t.batch, r);
  const int j = idx[(int64_t)kvh * idx_stride + r];
  if (j < 0 || j >= t.prompt_len[b]) {          // never read outside the sequence's prompt rows
    if (piece == 0) atomicOr(status, kStatusBadIndex);
    return;
  }
  const int64_t head_stride = is_v ? cv.v_head_stride : cv.k_head_stride;
  const int64_t row_stride = is_v ? cv.v_row_stride : cv.k_row_stride;
  const char* base = reinterpret_cast<const char*>(is_v ? cv.v : cv.k);
  const uint4* src = reinterpret_cast<const uint4*>(
      base + ((int64_t)kvh * head_stride + (int64_t)(t.cu_rows[b] + j) * row_stride) * elem_bytes);
  uint4* dst = (is_v ? v_out : k_out) + ((int64_t)kvh * kt + r) * kPieces;
  const uint4 val = __ldg(src + piece);
  __stcs(dst + piece, val);
}

}  // namespace

cudaError_t launch_compact(int dtype, const CacheDev& cv, const int32_t* idx, int64_t idx_stride,
                           void* k_out, void* v_out, const SeqTable& t, int n_kv_heads, int* status,
                           cudaStream_t s, LaunchLog* log) {
  log->begin(kKindCompact, s);
  const int kt = t.cu_keep[t.batch];
  if (dtype == DAPQ_BF16) {
    constexpr int P = kHeadDim * 2 / 16;
    const dim3 grid((unsigned)(((int64_t)kt * P + kCompactThreads - 1) / kCompactThreads), n_kv_heads, 2);
    launch_pdl(compact_kv_kernel<P>, grid, dim3(kCompactThreads), 0, s, 1, cv, 2, idx, idx_stride, (uint4*)k_out,
               (uint4*)v_out, t, status);
  } else {
    constexpr int P = kHeadDim * 4 / 16;
    const dim3 grid((unsigned)(((int64_t)kt * P + kCompactThreads - 1) / kCompactThreads), n_kv_heads, 2);
    launch_pdl(compact_kv_kernel<P>, grid, dim3(kCompactThreads), 0, s, 1, cv, 4, idx, idx_stride, (uint4*)k_out,
               (uint4*)v_out, t, status);
  }
  log->end(s);
  return cudaGetLastError();
}

}  // namespace dapq
