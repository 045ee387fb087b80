// Rotation of the pseudo queries to their decode positions (Section 4.1: the N synthetic
// tokens take positions L_p .. L_p+N-1, so their queries carry the positional encodings of
// the first N decoding steps).
//
// Grid (pseudo query i, sequence b, block of query heads); thread (c, hy) owns the channel
// pair of frequency c of one head: (c, c + d/2), or (2c, 2c + 1) for the interleaved layout.  The angle pos * theta_c is formed and reduced in double
// precision: at positions near 131k a float angle has only ~7 fractional bits, which alone
// would cost half of the scorer's error budget.  Each thread evaluates its own sincos (the
// table is tiny: B*N*64 angles), so no thread waits on another and the launch is one short
// wave of independent loads and stores.
#include <cuda_fp16.h>

#include "dapq_internal.cuh"

namespace dapq {
namespace {

constexpr int kHeadsPerBlock = 8;

template <typename T> __device__ __forceinline__ double to_double(T x);
template <> __device__ __forceinline__ double to_double<float>(float x) { return (double)x; }
template <> __device__ __forceinline__ double to_double<__nv_bfloat16>(__nv_bfloat16 x) {
  return (double)__bfloat162float(x);
}
template <> __device__ __forceinline__ double to_double<__half>(__half x) { return (double)__half2float(x); }
template <typename T> __device__ __forceinline__ T from_double(double x);
template <> __device__ __forceinline__ float from_double<float>(double x) { return (float)x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_double<__nv_bfloat16>(double x) {
  return __double2bfloat16(x);
}
// fp16 output (the query operand of the fp16 MMAs, stored times softmax scale * log2(e) so that the MMAs yield
// base-2 logits): values beyond the format's range saturate
template <> __device__ __forceinline__ __half from_double<__half>(double x) {
  return __double2half(fmin(fmax(x, -65504.0), 65504.0));
}

// kSplit: TO is bf16 and the rounding residual is stored as a second bf16 lo_offset elements on.
// ref (optional, bf16 caches): also the logit of every rotated query against the FIRST key of its
// sequence, ref.out[b, h, i] = out_scale * q_rot . K[h / G, cu_rows[b], :]: the first sweep of the
// tensor-core scorer measures every other logit of the row against it.
template <typename T, typename TO, bool kSplit>
__global__ void __launch_bounds__(kHeadDim / 2 * kHeadsPerBlock)
rope_pseudo_q_kernel(const T* __restrict__ q_pre, TO* __restrict__ q_rot,
                     const double* __restrict__ inv_freq, const __grid_constant__ SeqTable t,
                     int n_q_heads, int n_pseudo, int64_t lo_offset, int late_wait,
                     int interleaved, double out_scale, const RopeRef ref) {
  // late_wait: the kernel before this one in the stream neither writes q_pre nor still reads q_rot
  // (it is the compaction of the layer before), so the rotation runs beside it; the wait at the end
  // keeps this grid, and with it everything launched after it, ordered behind that kernel.
  pdl_trigger();
  if (!late_wait) pdl_wait();
  const int i = blockIdx.x, b = blockIdx.y, c = threadIdx.x;
  const int h = blockIdx.z * kHeadsPerBlock + threadIdx.y;
  const bool active = h < n_q_heads;
  constexpr int half = kHeadDim / 2;
  const int c0 = interleaved ? 2 * c : c, c1 = interleaved ? 2 * c + 1 : c + half;
  double r0 = 0.0, r1 = 0.0;
  if (active) {
    const size_t base = (((size_t)b * n_q_heads + h) * n_pseudo + i) * kHeadDim;
    const size_t e0 = base + c0, e1 = base + c1;
    const double lo = to_double<T>(q_pre[e0]);
    const double hi = to_double<T>(q_pre[e1]);
    const double ang = (double)(t.pos_start[b] + i) * inv_freq[c];
    double sn, cs;
    sincos(ang, &sn, &cs);
    r0 = (lo * cs - hi * sn) * out_scale;
    r1 = (hi * cs + lo * sn) * out_scale;
    const TO h0 = from_double<TO>(r0), h1 = from_double<TO>(r1);
    q_rot[e0] = h0;
    q_rot[e1] = h1;
    if (kSplit) {
      q_rot[lo_offset + e0] = from_double<TO>(r0 - to_double<TO>(h0));
      q_rot[lo_offset + e1] = from_double<TO>(r1 - to_double<TO>(h1));
    }
  }
  if (ref.out != nullptr) {                                     // (uniform over the grid)
    __shared__ float red[kHeadsPerBlock][2];
    float part = 0.f;
    if (active) {
      const __nv_bfloat16* k0 = ref.k + (int64_t)(h / ref.group) * ref.head_stride + (int64_t)t.cu_rows[b] * ref.row_stride;
      part = (float)r0 * __bfloat162float(k0[c0]) + (float)r1 * __bfloat162float(k0[c1]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    if ((c & 31) == 0) red[threadIdx.y][c >> 5] = part;         // the 64 threads of a head are two whole warps
    __syncthreads();
    if (active && c == 0) ref.out[((size_t)b * n_q_heads + h) * n_pseudo + i] = red[threadIdx.y][0] + red[threadIdx.y][1];
  }
  if (late_wait) pdl_wait();
}

}  // namespace

cudaError_t launch_rope(int dtype, int out_mode, int64_t lo_offset, const void* q_pre, void* q_rot,
                        const double* inv_freq_dev, const SeqTable& t, const Dims& dm, bool late_wait,
                        cudaStream_t s, LaunchLog* log, const RopeRef* ref_in) {
  RopeRef none = {nullptr, 0, 0, nullptr, 1};
  const RopeRef ref = (ref_in && out_mode == kRopeOutF16) ? *ref_in : none;
  const int lw = late_wait ? 1 : 0;
  log->begin(kKindRope, s);
  dim3 grid(dm.n_pseudo, t.batch, (dm.n_q_heads + kHeadsPerBlock - 1) / kHeadsPerBlock);
  dim3 block(kHeadDim / 2, kHeadsPerBlock);
  if (dtype == DAPQ_BF16 && out_mode == kRopeOutSplitBf16) {
    launch_pdl(rope_pseudo_q_kernel<__nv_bfloat16, __nv_bfloat16, true>, grid, block, 0, s, 1, (const __nv_bfloat16*)q_pre,
               (__nv_bfloat16*)q_rot, inv_freq_dev, t, dm.n_q_heads, dm.n_pseudo, lo_offset, lw, dm.rope_interleaved, 1.0, none);
  } else if (dtype == DAPQ_BF16 && out_mode == kRopeOutF16) {
    launch_pdl(rope_pseudo_q_kernel<__nv_bfloat16, __half, false>, grid, block, 0, s, 1, (const __nv_bfloat16*)q_pre,
               (__half*)q_rot, inv_freq_dev, t, dm.n_q_heads, dm.n_pseudo, 0, lw, dm.rope_interleaved, (double)dm.scale_log2e, ref);
  } else if (dtype == DAPQ_BF16 && out_mode == kRopeOutBf16) {
    launch_pdl(rope_pseudo_q_kernel<__nv_bfloat16, __nv_bfloat16, false>, grid, block, 0, s, 1, (const __nv_bfloat16*)q_pre,
               (__nv_bfloat16*)q_rot, inv_freq_dev, t, dm.n_q_heads, dm.n_pseudo, 0, lw, dm.rope_interleaved, 1.0, none);
  } else if (dtype == DAPQ_BF16) {
    launch_pdl(rope_pseudo_q_kernel<__nv_bfloat16, float, false>, grid, block, 0, s, 1, (const __nv_bfloat16*)q_pre,
               (float*)q_rot, inv_freq_dev, t, dm.n_q_heads, dm.n_pseudo, 0, lw, dm.rope_interleaved, 1.0, none);
  } else {
    launch_pdl(rope_pseudo_q_kernel<float, float, false>, grid, block, 0, s, 1, (const float*)q_pre, (float*)q_rot,
               inv_freq_dev, t, dm.n_q_heads, dm.n_pseudo, 0, lw, dm.rope_interleaved, 1.0, none);
  }
  log->end(s);
  return cudaGetLastError();
}

}  // namespace dapq
