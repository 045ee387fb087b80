// Pruning of the cache (Section 4.2: every key-value pair outside M_retain is discarded,
// and so is the whole synthetic segment).  A bit-exact gather of 256-byte (bf16) or
// 512-byte (fp32) rows: one thread per 16-byte piece of two rows, K and V in the same launch.
// Pure HBM traffic: rows_kept * row_bytes read + the same written, for K and for V.
#include "dapq_internal.cuh"

namespace dapq {
namespace {

constexpr int kCompactThreads = 256;

constexpr int kRowsPerThread = 2;

// One thread moves piece `piece` of kRowsPerThread kept rows, of K and of V: four independent 16-byte loads in
// flight per thread (the gather is bound by how many bytes the SMs keep in flight, not by instructions).
template <int kPieces>   // 16-byte pieces per row
__global__ void __launch_bounds__(kCompactThreads)
compact_kv_kernel(const CacheDev cv, int elem_bytes, const int32_t* __restrict__ idx, int64_t idx_stride,
                  uint4* __restrict__ k_out, uint4* __restrict__ v_out,
                  const __grid_constant__ SeqTable t, int* __restrict__ status) {
  pdl_trigger();                     // whatever follows may be set up (or, if it does not depend on this copy, run) beside it
  const int kt = t.cu_keep[t.batch];
  const int64_t gid = (int64_t)blockIdx.x * kCompactThreads + threadIdx.x;
  const int r0 = (int)(gid / kPieces) * kRowsPerThread, piece = (int)(gid % kPieces);
  const int kvh = blockIdx.y;
  int seg[kRowsPerThread];
#pragma unroll
  for (int i = 0; i < kRowsPerThread; ++i) seg[i] = r0 + i < kt ? find_segment(t.cu_keep, t.batch, r0 + i) : 0;
  pdl_wait();                        // the indices are written
  if (r0 >= kt) return;
  const char* k_base = reinterpret_cast<const char*>(cv.k);
  const char* v_base = reinterpret_cast<const char*>(cv.v);
  uint4 kv[kRowsPerThread], vv[kRowsPerThread];
  bool ok[kRowsPerThread];
  int j[kRowsPerThread];
#pragma unroll
  for (int i = 0; i < kRowsPerThread; ++i) j[i] = r0 + i < kt ? idx[(int64_t)kvh * idx_stride + r0 + i] : 0;
#pragma unroll
  for (int i = 0; i < kRowsPerThread; ++i) {
    ok[i] = r0 + i < kt && j[i] >= 0 && j[i] < t.prompt_len[seg[i]];   // never read outside the sequence's prompt rows
    if (ok[i]) {
      const int64_t row = t.cu_rows[seg[i]] + j[i];
      kv[i] = __ldg(reinterpret_cast<const uint4*>(k_base + ((int64_t)kvh * cv.k_head_stride + row * cv.k_row_stride) * elem_bytes) + piece);
      vv[i] = __ldg(reinterpret_cast<const uint4*>(v_base + ((int64_t)kvh * cv.v_head_stride + row * cv.v_row_stride) * elem_bytes) + piece);
    } else if (r0 + i < kt && piece == 0) {
      atomicOr(status, kStatusBadIndex);
    }
  }
#pragma unroll
  for (int i = 0; i < kRowsPerThread; ++i) {
    if (ok[i]) {
      const int64_t at = ((int64_t)kvh * kt + r0 + i) * kPieces + piece;
      __stcs(k_out + at, kv[i]);
      __stcs(v_out + at, vv[i]);
    }
  }
}

}  // namespace

cudaError_t launch_compact(int dtype, const CacheDev& cv, const int32_t* idx, int64_t idx_stride,
                           void* k_out, void* v_out, const SeqTable& t, int n_kv_heads, int* status,
                           cudaStream_t s, LaunchLog* log) {
  log->begin(kKindCompact, s);
  const int kt = t.cu_keep[t.batch];
  if (dtype == DAPQ_BF16) {
    constexpr int P = kHeadDim * 2 / 16;
    const dim3 grid((unsigned)(((int64_t)((kt + kRowsPerThread - 1) / kRowsPerThread) * P + kCompactThreads - 1) / kCompactThreads), n_kv_heads);
    launch_pdl(compact_kv_kernel<P>, grid, dim3(kCompactThreads), 0, s, 1, cv, 2, idx, idx_stride, (uint4*)k_out,
               (uint4*)v_out, t, status);
  } else {
    constexpr int P = kHeadDim * 4 / 16;
    const dim3 grid((unsigned)(((int64_t)((kt + kRowsPerThread - 1) / kRowsPerThread) * P + kCompactThreads - 1) / kCompactThreads), n_kv_heads);
    launch_pdl(compact_kv_kernel<P>, grid, dim3(kCompactThreads), 0, s, 1, cv, 4, idx, idx_stride, (uint4*)k_out,
               (uint4*)v_out, t, status);
  }
  log->end(s);
  return cudaGetLastError();
}

}  // namespace dapq
