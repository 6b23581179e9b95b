// Stage 1 on CUDA cores (fp32 arithmetic): attention column sums (Algorithm 1 of the paper,
// "attention weights" and "normalized attention score" steps).  Serves fp32 inputs and shapes the
// tensor-core kernels do not cover (bf16 and fp16 inputs are widened on load); the S x S matrix is never stored.
//
//   lse_rows_kernel   one warp per query row j: lanes take keys t, t+32, ..; each lane keeps an
//                     online (max, sum) pair in the log2 domain; lse2(j) = log2 sum_t 2^(s2(j,t))
//                     with s2 = q.k * scale * log2(e).
//   colsum_kernel     one warp per key t: lanes take queries j, j+32, ..; accumulates
//                     2^(s2(j,t) - lse2(j)) = A(j,t) and reduces over the warp.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.cuh"

namespace kvc {

namespace {

constexpr int kWarpsPerBlock = 4;
constexpr int kMaxD = 256;

template <typename T>
__device__ __forceinline__ void load8(const T* p, float (&v)[8]);

template <>
__device__ __forceinline__ void load8<float>(const float* p, float (&v)[8]) {
  const float4 a = __ldg(reinterpret_cast<const float4*>(p));
  const float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

template <>
__device__ __forceinline__ void load8<__nv_bfloat16>(const __nv_bfloat16* p, float (&v)[8]) {
  const uint4 r = __ldg(reinterpret_cast<const uint4*>(p));
  const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}

template <>
__device__ __forceinline__ void load8<__half>(const __half* p, float (&v)[8]) {
  const uint4 r = __ldg(reinterpret_cast<const uint4*>(p));
  const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
    v[2 * i] = f.x;
    v[2 * i + 1] = f.y;
  }
}

template <typename T>
__device__ __forceinline__ float dot_row(const float* __restrict__ a_sh, const T* __restrict__ b, int D) {
  float acc = 0.f;
  for (int d = 0; d < D; d += 8) {
    float v[8];
    load8<T>(b + d, v);
#pragma unroll
    for (int i = 0; i < 8; ++i) acc = fmaf(a_sh[d + i], v[i], acc);
  }
  return acc;
}

template <typename T>
__device__ __forceinline__ void stage_row(float* sh, const T* row, int D, int lane) {
  for (int d = lane * 8; d < D; d += 32 * 8) {
    float v[8];
    load8<T>(row + d, v);
#pragma unroll
    for (int i = 0; i < 8; ++i) sh[d + i] = v[i];
  }
  __syncwarp();
}

template <typename T>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
lse_rows_kernel(Shape s, TensorView Q, TensorView K, float scale_log2, float* __restrict__ lse2,
                float* __restrict__ lse_out) {
  __shared__ float q_sh[kWarpsPerBlock][kMaxD];
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const long long row = (long long)blockIdx.x * kWarpsPerBlock + wib;     // (layer, head, token)
  if (row >= (long long)s.n_layers * s.Hq * s.T) return;
  const int tok = (int)(row % s.T);
  const int h = (int)((row / s.T) % s.Hq);
  const int layer = (int)(row / ((long long)s.T * s.Hq));
  const int seq = seq_of_token(s.cu_seqlens, s.n_seqs, tok);
  const int t0 = __ldg(s.cu_seqlens + seq), t1 = __ldg(s.cu_seqlens + seq + 1);
  const int t_end = s.causal ? tok + 1 : t1;
  const int ws = (s.window > 0 && t1 - t0 > s.window) ? t1 - t0 - s.window : 0;   // first voting query of the sequence
  if (tok - t0 < ws) return;                       // this query does not vote: its log-sum-exp is not needed

  const T* q = static_cast<const T*>(Q.ptr) + layer * Q.sl + (long long)tok * Q.st + h * Q.sh;
  const T* kbase = static_cast<const T*>(K.ptr) + layer * K.sl + (h / s.G) * K.sh;
  stage_row<T>(q_sh[wib], q, s.D, lane);

  float m = -INFINITY, sum = 0.f;
  for (int t = t0 + lane; t < t_end; t += 32) {
    const float x = dot_row<T>(q_sh[wib], kbase + (long long)t * K.st, s.D) * scale_log2;
    if (x > m) { sum = sum * exp2f(m - x) + 1.f; m = x; } else { sum += exp2f(x - m); }
  }
  float big = m;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) big = fmaxf(big, __shfl_xor_sync(0xFFFFFFFFu, big, d));
  float part = (m == -INFINITY) ? 0.f : sum * exp2f(m - big);
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, d);
  if (lane == 0) {
    const float v = big + log2f(part);
    lse2[row] = v;
    if (lse_out) lse_out[row] = v * 0.69314718055994530942f;
  }
}

template <typename T>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
colsum_kernel(Shape s, TensorView Q, TensorView K, float scale_log2, const float* __restrict__ lse,
              float lse_mul, float* __restrict__ scores, int normalize) {
  __shared__ float k_sh[kWarpsPerBlock][kMaxD];
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const long long col = (long long)blockIdx.x * kWarpsPerBlock + wib;     // (layer, head, token)
  if (col >= (long long)s.n_layers * s.Hq * s.T) return;
  const int tok = (int)(col % s.T);
  const int h = (int)((col / s.T) % s.Hq);
  const int layer = (int)(col / ((long long)s.T * s.Hq));
  const int seq = seq_of_token(s.cu_seqlens, s.n_seqs, tok);
  const int t0 = __ldg(s.cu_seqlens + seq), t1 = __ldg(s.cu_seqlens + seq + 1);
  const int ws = (s.window > 0 && t1 - t0 > s.window) ? t1 - t0 - s.window : 0;   // first voting query of the sequence
  const int j_begin = max(s.causal ? tok : t0, t0 + ws);

  const T* k = static_cast<const T*>(K.ptr) + layer * K.sl + (long long)tok * K.st + (h / s.G) * K.sh;
  const T* qbase = static_cast<const T*>(Q.ptr) + layer * Q.sl + h * Q.sh;
  const float* lse_row = lse + ((long long)layer * s.Hq + h) * s.T;
  stage_row<T>(k_sh[wib], k, s.D, lane);

  float acc = 0.f;
  for (int j = j_begin + lane; j < t1; j += 32) {
    const float x = dot_row<T>(k_sh[wib], qbase + (long long)j * Q.st, s.D) * scale_log2;
    acc += exp2f(x - __ldg(lse_row + j) * lse_mul);
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, d);
  if (lane == 0) scores[col] = normalize ? acc / (float)(t1 - t0 - ws) : acc;
}

// Decode step: every sequence has one new query (its last token); the query's attention row over the sequence's
// cached keys is added to the running scores.  One block per (layer, sequence, KV head); threads stride over the
// tokens and serve up to kDecodeHeads query heads of the KV group from one read of a key row.  Pass 1 keeps an
// online (max, sum) per thread and head and reduces it over the block, pass 2 recomputes the logits and adds
// 2^(x - lse2) to scores (each token is owned by one thread: no atomics).
constexpr int kDecodeThreads = 256;
constexpr int kDecodeHeads = 4;

template <typename T>
__device__ __forceinline__ void dot_rows(const float (*q_sh)[kMaxD], const T* __restrict__ krow, int D, int n_heads,
                                         float (&acc)[kDecodeHeads]) {
#pragma unroll
  for (int g = 0; g < kDecodeHeads; ++g) acc[g] = 0.f;
  for (int d = 0; d < D; d += 8) {
    float v[8];
    load8<T>(krow + d, v);
#pragma unroll
    for (int g = 0; g < kDecodeHeads; ++g)
      if (g < n_heads) {
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[g] = fmaf(q_sh[g][d + i], v[i], acc[g]);
      }
  }
}

template <typename T>
__global__ void __launch_bounds__(kDecodeThreads)
decode_update_kernel(Shape s, TensorView Qn, TensorView K, float scale_log2, float* __restrict__ scores) {
  __shared__ float q_sh[kDecodeHeads][kMaxD];
  __shared__ float red_m[kDecodeHeads][kDecodeThreads / 32], red_s[kDecodeHeads][kDecodeThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, wib = tid >> 5;
  const int hk = blockIdx.x % s.Hkv;
  const int seq = (blockIdx.x / s.Hkv) % s.n_seqs;
  const int layer = blockIdx.x / (s.Hkv * s.n_seqs);
  const int t0 = __ldg(s.cu_seqlens + seq), t1 = __ldg(s.cu_seqlens + seq + 1);
  if (t1 <= t0) return;
  const T* kbase = static_cast<const T*>(K.ptr) + layer * K.sl + hk * K.sh;

  for (int g0 = 0; g0 < s.G; g0 += kDecodeHeads) {                // the KV group's query heads, a few at a time
    const int n_heads = min(kDecodeHeads, s.G - g0);
    const int h0 = hk * s.G + g0;
    __syncthreads();                                              // q_sh / red_* of the previous round are done with
    for (int e = tid * 8; e < n_heads * s.D; e += kDecodeThreads * 8) {
      const int g = e / s.D, d = e - g * s.D;
      const T* q = static_cast<const T*>(Qn.ptr) + layer * Qn.sl + (long long)seq * Qn.st + (h0 + g) * Qn.sh;
      float v[8];
      load8<T>(q + d, v);
#pragma unroll
      for (int i = 0; i < 8; ++i) q_sh[g][d + i] = v[i];
    }
    __syncthreads();

    float m[kDecodeHeads], sum[kDecodeHeads];
#pragma unroll
    for (int g = 0; g < kDecodeHeads; ++g) { m[g] = -INFINITY; sum[g] = 0.f; }
    for (int t = t0 + tid; t < t1; t += kDecodeThreads) {
      float x[kDecodeHeads];
      dot_rows<T>(q_sh, kbase + (long long)t * K.st, s.D, n_heads, x);
#pragma unroll
      for (int g = 0; g < kDecodeHeads; ++g) {
        const float xs = x[g] * scale_log2;
        if (xs > m[g]) { sum[g] = sum[g] * exp2f(m[g] - xs) + 1.f; m[g] = xs; } else { sum[g] += exp2f(xs - m[g]); }
      }
    }
#pragma unroll
    for (int g = 0; g < kDecodeHeads; ++g) {
      float big = m[g];
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) big = fmaxf(big, __shfl_xor_sync(0xFFFFFFFFu, big, d));
      float part = (m[g] == -INFINITY) ? 0.f : sum[g] * exp2f(m[g] - big);
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, d);
      if (lane == 0) { red_m[g][wib] = big; red_s[g][wib] = part; }
    }
    __syncthreads();
    float lse2[kDecodeHeads];
#pragma unroll
    for (int g = 0; g < kDecodeHeads; ++g) {
      float all_m = -INFINITY, all_s = 0.f;
      for (int w = 0; w < kDecodeThreads / 32; ++w) all_m = fmaxf(all_m, red_m[g][w]);
      for (int w = 0; w < kDecodeThreads / 32; ++w)
        all_s += red_m[g][w] == -INFINITY ? 0.f : red_s[g][w] * exp2f(red_m[g][w] - all_m);
      lse2[g] = all_m + log2f(all_s);
    }

    for (int t = t0 + tid; t < t1; t += kDecodeThreads) {
      float x[kDecodeHeads];
      dot_rows<T>(q_sh, kbase + (long long)t * K.st, s.D, n_heads, x);
#pragma unroll
      for (int g = 0; g < kDecodeHeads; ++g)
        if (g < n_heads) scores[((long long)layer * s.Hq + h0 + g) * s.T + t] += exp2f(x[g] * scale_log2 - lse2[g]);
    }
  }
}

template <typename T>
int run_decode(const Shape& s, const TensorView& Qn, const TensorView& K, float scale_log2, float* scores,
               cudaStream_t stream) {
  const long long blocks = (long long)s.n_layers * s.n_seqs * s.Hkv;
  if (blocks > 0x7FFFFFFFLL) return KVCRUSH_ERR_UNSUPPORTED;
  decode_update_kernel<T><<<(unsigned)blocks, kDecodeThreads, 0, stream>>>(s, Qn, K, scale_log2, scores);
  return check_launch();
}

template <typename T>
int run(const Shape& s, const TensorView& Q, const TensorView& K, float scale_log2, const float* lse_in,
        float lse_in_mul, float* lse2_ws, float* scores, float* lse_out, int normalize, cudaStream_t stream) {
  const long long rows = (long long)s.n_layers * s.Hq * s.T;
  if (rows == 0) return KVCRUSH_OK;
  const long long blocks = (rows + kWarpsPerBlock - 1) / kWarpsPerBlock;
  if (blocks > 0x7FFFFFFFLL) return KVCRUSH_ERR_UNSUPPORTED;
  const float* lse = lse_in;
  float mul = lse_in_mul;
  if (!lse_in) {
    lse_rows_kernel<T><<<(unsigned)blocks, kWarpsPerBlock * 32, 0, stream>>>(s, Q, K, scale_log2, lse2_ws, lse_out);
    if (check_launch() != KVCRUSH_OK) return KVCRUSH_ERR_CUDA;
    lse = lse2_ws;
    mul = 1.f;
  }
  colsum_kernel<T><<<(unsigned)blocks, kWarpsPerBlock * 32, 0, stream>>>(s, Q, K, scale_log2, lse, mul, scores,
                                                                          normalize);
  return check_launch();
}

}  // namespace

int launch_score_simt(const Shape& s, const TensorView& Q, const TensorView& K, float scale_log2,
                      const float* lse_in, float lse_in_mul, float* lse2_ws, float* scores, float* lse_out,
                      int normalize, int32_t* /*status*/, cudaStream_t stream) {
  if (s.D > kMaxD || s.D % 8 != 0) return KVCRUSH_ERR_UNSUPPORTED;
  if (Q.dtype == KVCRUSH_FP32)
    return run<float>(s, Q, K, scale_log2, lse_in, lse_in_mul, lse2_ws, scores, lse_out, normalize, stream);
  if (Q.dtype == KVCRUSH_BF16)
    return run<__nv_bfloat16>(s, Q, K, scale_log2, lse_in, lse_in_mul, lse2_ws, scores, lse_out, normalize, stream);
  if (Q.dtype == KVCRUSH_FP16)
    return run<__half>(s, Q, K, scale_log2, lse_in, lse_in_mul, lse2_ws, scores, lse_out, normalize, stream);
  return KVCRUSH_ERR_UNSUPPORTED;
}

int launch_score_decode(const Shape& s, const TensorView& Q_new, const TensorView& K, float scale_log2, float* scores,
                        cudaStream_t stream) {
  if (s.D > kMaxD || s.D % 8 != 0) return KVCRUSH_ERR_UNSUPPORTED;
  if (s.T == 0) return KVCRUSH_OK;
  if (Q_new.dtype == KVCRUSH_FP32) return run_decode<float>(s, Q_new, K, scale_log2, scores, stream);
  if (Q_new.dtype == KVCRUSH_BF16) return run_decode<__nv_bfloat16>(s, Q_new, K, scale_log2, scores, stream);
  if (Q_new.dtype == KVCRUSH_FP16) return run_decode<__half>(s, Q_new, K, scale_log2, scores, stream);
  return KVCRUSH_ERR_UNSUPPORTED;
}

}  // namespace kvc
