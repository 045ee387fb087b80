// Importance scoring on the CUDA cores (Section 4.2, Eq. 4):
//   S(j) = sum_i Attention(q_i, k_j),  Attention = softmax(q K^T / sqrt(d_k)),
// summed over the query heads of a GQA group.  This is the general path: any N <= 128,
// fp32 or bf16 storage, fp32 arithmetic throughout.  It serves the fp32 caches (whose
// precision a bf16 tensor-core product would not keep) and every shape the tensor-core
// path does not take.
//
// Column sums of a row-normalised matrix need every row's normaliser before any column
// can be summed, so the keys are swept twice:
//   sweep 1  per (chunk of keys, query head, pseudo query): running max and sum of exp
//            -> partials, merged into one log-sum-exp per pseudo query;
//   sweep 2  P_ij = exp(s_ij - lse_i), summed over the N queries and the G heads.
// Logits are kept in base 2 (s * scale * log2 e) so that every exponential is one ex2.
// All reductions run in a fixed order: results are bit-identical from run to run.
#include <math_constants.h>

#include "dapq_internal.cuh"

namespace dapq {
namespace {

constexpr int kTileKeys = 64;     // keys per shared-memory tile
constexpr int kPad = 132;         // fp32 words per shared-memory row (128 + 4: conflict-free float4)
constexpr int kThreads = 256;     // 16 (query rows) x 16 (key columns)

template <typename T> struct Chunk16;
template <> struct Chunk16<float> {
  static constexpr int kElems = 4;
  static __device__ __forceinline__ void load(const float* p, float* out) {
    const float4 v = __ldg(reinterpret_cast<const float4*>(p));
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
  }
};
template <> struct Chunk16<__nv_bfloat16> {
  static constexpr int kElems = 8;
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float* out) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      out[2 * e] = __uint_as_float(w[e] << 16);
      out[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
    }
  }
};

// Copy n_tile rows of 128 elements into fp32 shared memory; rows >= n_valid become zero.
template <typename T>
__device__ __forceinline__ void stage_rows(float* dst, const T* src, int64_t row_stride,
                                           int n_valid, int n_tile) {
  constexpr int E = Chunk16<T>::kElems;
  constexpr int CPR = kHeadDim / E;
  for (int x = threadIdx.x; x < n_tile * CPR; x += kThreads) {
    const int r = x / CPR, c = x % CPR;
    float vals[E];
    if (r < n_valid) {
      Chunk16<T>::load(src + (int64_t)r * row_stride + c * E, vals);
    } else {
#pragma unroll
      for (int e = 0; e < E; ++e) vals[e] = 0.f;
    }
    float* d = dst + r * kPad + c * E;
#pragma unroll
    for (int e = 0; e < E; e += 4)
      *reinterpret_cast<float4*>(d + e) = make_float4(vals[e], vals[e + 1], vals[e + 2], vals[e + 3]);
  }
}

template <int R>
constexpr size_t fma_smem_bytes() {
  return sizeof(float) * (size_t)(16 * R * kPad + kTileKeys * kPad + 8 * kTileKeys + kChunkKeys + 16 * R);
}

// grid (n_chunks, H_kv) in sweep 2, which sums over the G heads of the group in a fixed order;
// (n_chunks, H_kv, G) in sweep 1, whose partials are per head.  A chunk holds ct.chunk_tiles
// prompt keys (64 .. kChunkKeys, chosen per call).  Thread (ty, tx) owns query rows ty + 16 r
// (r < R) and the keys kk * 16 + tx (kk < 4) of each 64-key tile.
template <typename TQ, typename T, int R, bool kSweep2>
__global__ void __launch_bounds__(kThreads)
score_fma_kernel(const TQ* __restrict__ q_rot, const CacheDev cv, const __grid_constant__ SeqTable t,
                 const __grid_constant__ ChunkTable ct, const Dims dm, float2* __restrict__ part, const float* __restrict__ lse2,
                 float* __restrict__ scores, int64_t score_stride, float* __restrict__ syn_mass) {
  extern __shared__ __align__(16) float smem[];
  float* Qs = smem;                          // [16 R][kPad]
  float* Ks = Qs + 16 * R * kPad;            // [64][kPad]
  float* red = Ks + kTileKeys * kPad;        // [8 warps][64]
  float* colacc = red + 8 * kTileKeys;       // [kChunkKeys]
  float* lse_s = colacc + kChunkKeys;        // [16 R]

  const int chunk = blockIdx.x, kvh = blockIdx.y, tid = threadIdx.x;
  const int b = find_segment(ct.cu_chunk, t.batch, chunk);
  const int c = chunk - ct.cu_chunk[b], chunk_keys = ct.chunk_tiles;
  const int L = t.prompt_len[b], N = dm.n_pseudo, G = dm.group, Hq = dm.n_q_heads;
  const bool syn = (c == ct.cu_chunk[b + 1] - ct.cu_chunk[b] - 1);
  const int key_begin = syn ? L : c * chunk_keys;
  const int key_end = syn ? L + N : min(L, key_begin + chunk_keys);
  if (kSweep2 && syn && syn_mass == nullptr) return;

  const T* kbase = reinterpret_cast<const T*>(cv.k) + (int64_t)kvh * cv.k_head_stride +
                   (int64_t)t.cu_rows[b] * cv.k_row_stride;
  const int tx = tid & 15, ty = tid >> 4, lane = tid & 31, warp = tid >> 5;

  if (kSweep2) {
    for (int x = tid; x < kChunkKeys; x += kThreads) colacc[x] = 0.f;
  }

  const int g_begin = kSweep2 ? 0 : (int)blockIdx.z, g_end = kSweep2 ? G : g_begin + 1;
  for (int g = g_begin; g < g_end; ++g) {
    const int h = kvh * G + g;
    __syncthreads();                                        // Qs, lse_s, colacc free
    stage_rows<TQ>(Qs, q_rot + ((int64_t)b * Hq + h) * N * kHeadDim, kHeadDim, N, 16 * R);
    if (kSweep2) {
      for (int x = tid; x < 16 * R; x += kThreads)
        lse_s[x] = (x < N) ? lse2[((int64_t)b * Hq + h) * N + x] : 0.f;
    }
    float m[R], z[R];
#pragma unroll
    for (int r = 0; r < R; ++r) { m[r] = -CUDART_INF_F; z[r] = 0.f; }

    for (int k0 = key_begin; k0 < key_end; k0 += kTileKeys) {
      __syncthreads();                                      // Ks free; Qs visible
      stage_rows<T>(Ks, kbase + (int64_t)k0 * cv.k_row_stride, cv.k_row_stride,
                    min(kTileKeys, key_end - k0), kTileKeys);
      __syncthreads();

      float acc[R][4];
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) acc[r][kk] = 0.f;
#pragma unroll 4
      for (int dd = 0; dd < kHeadDim; dd += 4) {
        float4 kv[4];
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          kv[kk] = *reinterpret_cast<const float4*>(Ks + (kk * 16 + tx) * kPad + dd);
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const float4 qv = *reinterpret_cast<const float4*>(Qs + (ty + 16 * r) * kPad + dd);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            acc[r][kk] = fmaf(qv.x, kv[kk].x, acc[r][kk]);
            acc[r][kk] = fmaf(qv.y, kv[kk].y, acc[r][kk]);
            acc[r][kk] = fmaf(qv.z, kv[kk].z, acc[r][kk]);
            acc[r][kk] = fmaf(qv.w, kv[kk].w, acc[r][kk]);
          }
        }
      }

      // base-2 logits; a key is visible to query i if it is a prompt key or synthetic key <= i
      float colsum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const int i = ty + 16 * r;
        float s[4];
        float tmax = -CUDART_INF_F;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          const int j = k0 + kk * 16 + tx;
          const bool vis = (j < key_end) && (j <= L + i) && (i < N);
          s[kk] = vis ? acc[r][kk] * dm.scale_log2e : -CUDART_INF_F;
          tmax = fmaxf(tmax, s[kk]);
        }
        if (!kSweep2) {
#pragma unroll
          for (int o = 1; o < 16; o <<= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
          const float m_new = fmaxf(m[r], tmax);
          float sum = 0.f;
          if (m_new > -CUDART_INF_F) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) sum += exp2f(s[kk] - m_new);
          }
#pragma unroll
          for (int o = 1; o < 16; o <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
          if (m_new > -CUDART_INF_F) {
            z[r] = z[r] * exp2f(m[r] - m_new) + sum;
            m[r] = m_new;
          }
        } else {
          const float l2 = lse_s[i];
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) colsum[kk] += exp2f(s[kk] - l2);   // exp2(-inf) = 0
        }
      }
      if (kSweep2) {
        // sum over the 16 row groups: the two of this warp by shuffle, the 8 warps through smem
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          colsum[kk] += __shfl_xor_sync(0xffffffffu, colsum[kk], 16);
          if (lane < 16) red[warp * kTileKeys + kk * 16 + tx] = colsum[kk];
        }
        __syncthreads();
        if (tid < kTileKeys) {
          float a = 0.f;
#pragma unroll
          for (int w = 0; w < 8; ++w) a += red[w * kTileKeys + tid];
          colacc[k0 - key_begin + tid] += a;
        }
      }
    }

    if (!kSweep2) {
      if (tx == 0) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const int i = ty + 16 * r;
          if (i < N) part[((int64_t)chunk * Hq + h) * N + i] = make_float2(m[r], z[r]);
        }
      }
    } else if (syn) {
      // attention mass of this head on its synthetic keys, summed in a fixed order
      __syncthreads();
      if (warp == 0) {
        float a = 0.f;
        for (int x = lane; x < N; x += 32) a += colacc[x];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        if (lane == 0) syn_mass[(int64_t)b * Hq + h] = a;
      }
      __syncthreads();
      for (int x = tid; x < kChunkKeys; x += kThreads) colacc[x] = 0.f;
    }
  }

  if (kSweep2 && !syn) {
    __syncthreads();
    float* out = scores + (int64_t)kvh * score_stride + t.cu_prompt[b] + key_begin;
    for (int x = tid; x < key_end - key_begin; x += kThreads) out[x] = colacc[x];
  }
}

// Merge the per-chunk (max, sum) partials of one pseudo query into its base-2 log-sum-exp.
__global__ void lse_merge_kernel(const float2* __restrict__ part, const __grid_constant__ SeqTable t,
                                 const __grid_constant__ ChunkTable ct, int n_q_heads, int n_pseudo, float* __restrict__ lse2,
                                 float* __restrict__ lse_out) {
  const int x = blockIdx.x * blockDim.x + threadIdx.x;
  const int per_seq = n_q_heads * n_pseudo;
  if (x >= t.batch * per_seq) return;
  const int b = x / per_seq, hi = x % per_seq;
  float mx = -CUDART_INF_F;
  for (int c = ct.cu_chunk[b]; c < ct.cu_chunk[b + 1]; ++c)
    mx = fmaxf(mx, part[(int64_t)c * per_seq + hi].x);
  float z = 0.f;
  for (int c = ct.cu_chunk[b]; c < ct.cu_chunk[b + 1]; ++c) {
    const float2 p = part[(int64_t)c * per_seq + hi];
    z += p.y * exp2f(p.x - mx);
  }
  const float l2 = mx + log2f(z);
  lse2[x] = l2;
  if (lse_out) lse_out[x] = l2 * 0.6931471805599453f;
}

// Caller-supplied natural-log lse -> base 2.
__global__ void lse_import_kernel(const float* __restrict__ lse_in, int n, float* __restrict__ lse2,
                                  float* __restrict__ lse_out) {
  const int x = blockIdx.x * blockDim.x + threadIdx.x;
  if (x >= n) return;
  lse2[x] = lse_in[x] * 1.4426950408889634f;
  if (lse_out) lse_out[x] = lse_in[x];
}

template <typename TQ, typename T, int R>
cudaError_t run_fma(const void* q_rot, const CacheDev& cv, const SeqTable& t, const Dims& dm,
                    const float* lse_in, float2* part, int64_t max_chunks, int n_sm, float* lse2, float* scores,
                    int64_t score_stride, float* lse_out, float* syn_mass, cudaStream_t s,
                    LaunchLog* log) {
  constexpr size_t smem = fma_smem_bytes<R>();
  auto k1 = score_fma_kernel<TQ, T, R, false>;
  auto k2 = score_fma_kernel<TQ, T, R, true>;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  // Keys per chunk: the largest of 512 .. 64 that gives every SM two CTAs in sweep 2, else the
  // smallest whose partials fit the caller's buffer (512 always fits: the callers check it).
  ChunkTable ct;
  ct.chunk_tiles = kChunkKeys;
  int32_t n_chunks = 0;
  for (int ck = kChunkKeys; ck >= kTileKeys; ck >>= 1) {
    int64_t n = 0;
    for (int b = 0; b < t.batch; ++b) n += (t.prompt_len[b] + ck - 1) / ck + 1;
    if (ck < kChunkKeys && n > max_chunks) break;
    ct.chunk_tiles = ck;
    n_chunks = (int32_t)n;
    if (n * dm.n_kv_heads >= 2LL * n_sm) break;
  }
  for (int b = 0, n = 0; b <= t.batch; ++b) {
    ct.cu_chunk[b] = n;
    if (b < t.batch) n += (t.prompt_len[b] + ct.chunk_tiles - 1) / ct.chunk_tiles + 1;
  }
  ct.n_chunks = n_chunks;
  const dim3 grid(n_chunks, dm.n_kv_heads), grid1(n_chunks, dm.n_kv_heads, dm.group);
  const int n_lse = t.batch * dm.n_q_heads * dm.n_pseudo;
  if (lse_in == nullptr) {
    log->begin(kKindSweep1, s);
    k1<<<grid1, kThreads, smem, s>>>((const TQ*)q_rot, cv, t, ct, dm, part, nullptr, nullptr, 0, nullptr);
    log->end(s);
    log->begin(kKindLseMerge, s);
    lse_merge_kernel<<<(n_lse + 127) / 128, 128, 0, s>>>(part, t, ct, dm.n_q_heads, dm.n_pseudo, lse2, lse_out);
    log->end(s);
  } else {
    log->begin(kKindLseMerge, s);
    lse_import_kernel<<<(n_lse + 127) / 128, 128, 0, s>>>(lse_in, n_lse, lse2, lse_out);
    log->end(s);
  }
  log->begin(kKindSweep2, s);
  k2<<<grid, kThreads, smem, s>>>((const TQ*)q_rot, cv, t, ct, dm, nullptr, lse2, scores, score_stride, syn_mass);
  log->end(s);
  return cudaGetLastError();
}

template <typename TQ, typename T>
cudaError_t run_fma_n(const void* q_rot, const CacheDev& cv, const SeqTable& t, const Dims& dm,
                      const float* lse_in, float2* part, int64_t max_chunks, int n_sm, float* lse2, float* scores,
                      int64_t score_stride, float* lse_out, float* syn_mass, cudaStream_t s,
                      LaunchLog* log) {
  const int n = dm.n_pseudo;
  if (n <= 16) return run_fma<TQ, T, 1>(q_rot, cv, t, dm, lse_in, part, max_chunks, n_sm, lse2, scores, score_stride, lse_out, syn_mass, s, log);
  if (n <= 32) return run_fma<TQ, T, 2>(q_rot, cv, t, dm, lse_in, part, max_chunks, n_sm, lse2, scores, score_stride, lse_out, syn_mass, s, log);
  if (n <= 64) return run_fma<TQ, T, 4>(q_rot, cv, t, dm, lse_in, part, max_chunks, n_sm, lse2, scores, score_stride, lse_out, syn_mass, s, log);
  return run_fma<TQ, T, 8>(q_rot, cv, t, dm, lse_in, part, max_chunks, n_sm, lse2, scores, score_stride, lse_out, syn_mass, s, log);
}

}  // namespace

namespace {
template <typename TQ, typename T, int R>
cudaError_t preload_fma() {
  constexpr size_t smem = fma_smem_bytes<R>();
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(score_fma_kernel<TQ, T, R, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  return cudaFuncSetAttribute(score_fma_kernel<TQ, T, R, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}
template <typename TQ, typename T>
cudaError_t preload_fma_n() {
  cudaError_t e;
  if ((e = preload_fma<TQ, T, 1>()) != cudaSuccess) return e;
  if ((e = preload_fma<TQ, T, 2>()) != cudaSuccess) return e;
  if ((e = preload_fma<TQ, T, 4>()) != cudaSuccess) return e;
  return preload_fma<TQ, T, 8>();
}
}  // namespace

// Touch every kernel that launch_score_fma can pick for storage type == query type, so that the device
// code of all of them is resident on the current device afterwards (with lazy module loading a kernel's
// code is brought to the device, and device memory taken for it, at its first use).
cudaError_t score_fma_preload() {
  cudaError_t e;
  if ((e = preload_fma_n<__nv_bfloat16, __nv_bfloat16>()) != cudaSuccess) return e;
  if ((e = preload_fma_n<float, float>()) != cudaSuccess) return e;
  cudaFuncAttributes fa;
  if ((e = cudaFuncGetAttributes(&fa, lse_merge_kernel)) != cudaSuccess) return e;
  return cudaFuncGetAttributes(&fa, lse_import_kernel);
}

cudaError_t launch_score_fma(int dtype, int q_dtype, const void* q_rot, const CacheDev& cv, const SeqTable& t,
                             const Dims& dm, const float* lse_in, float2* part, int64_t max_chunks, int n_sm,
                             float* lse2, float* scores, int64_t score_stride, float* lse_out, float* syn_mass,
                             cudaStream_t s, LaunchLog* log) {
  if (dtype == DAPQ_BF16 && q_dtype == DAPQ_BF16)
    return run_fma_n<__nv_bfloat16, __nv_bfloat16>(q_rot, cv, t, dm, lse_in, part, max_chunks, n_sm, lse2, scores, score_stride, lse_out, syn_mass, s, log);
  if (dtype == DAPQ_BF16)
    return run_fma_n<float, __nv_bfloat16>(q_rot, cv, t, dm, lse_in, part, max_chunks, n_sm, lse2, scores, score_stride, lse_out, syn_mass, s, log);
  return run_fma_n<float, float>(q_rot, cv, t, dm, lse_in, part, max_chunks, n_sm, lse2, scores, score_stride, lse_out, syn_mass, s, log);
}

}  // namespace dapq
