// Stage 2: per-head thresholds and packed binary signatures (Algorithm 1 and Sec. 3.1 of the paper).
//
//   theta_select_kernel       theta = keep-th largest score of one (layer, sequence, head) row of up to 32768
//                             tokens: the row is read once into registers as order-preserving 32-bit keys, and
//                             the k-th largest is found by 12-bit radix histograms over (key - smallest key),
//                             starting at the top bit in which the row's keys differ at all; one warp ranks the
//                             last few candidates directly.  Usually one histogram pass.
//   theta_stream_kernel       the same result for longer rows: MSB-first radix select (4 sweeps of 8 bits) that
//                             re-reads the row from memory (or from a shared-memory copy) in every sweep.
//   signature_pack_kernel     one block per (layer, 128 tokens): stages the [heads][tokens] tile of scores in shared
//                             memory with 16-byte row loads, then one thread per token compares its score of every
//                             head with that head's threshold and packs the bits; from the same tile it can add up
//                             the token's importance I(t) in float64, in the fixed order stage 3 defines, which
//                             saves stage 3 its own pass over the scores.
#include "select_common.cuh"

namespace kvc {

namespace {

constexpr int kSelectThreads = 512;
constexpr int kThetaBits = 12;                 // radix digit of theta_select_kernel
constexpr int kThetaBins = 1 << kThetaBits;

// float -> uint32 such that a < b  <=>  key(a) < key(b) (for non-NaN values)
__device__ __forceinline__ uint32_t order_key(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_to_float(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

// kT threads, each holding up to kItems keys of the row: rows of up to kT * kItems tokens.  kMinB: resident blocks per
// SM the kernel is compiled for.  The kernel is a chain of short dependent steps, so what counts is how many rows an
// SM works on at once and how many threads share a row: measured for 1024 rows of 8192 scores, 512 threads x 16 keys
// at 4 blocks per SM (32 registers, a few spilled words) 16.2 us, 256 x 32 at 4 per SM 17.9 us, 512 x 16 at 2 per SM
// 20.3 us, 1024 x 8 at 2 per SM 19.7 us, 128 x 64 23.7 us.
template <int kT, int kItems, int kMinB>
__global__ void __launch_bounds__(kT, kMinB)
theta_select_kernel(Shape s, const float* __restrict__ scores, const int32_t* __restrict__ sig_keep,
                    float* __restrict__ theta) {
  __shared__ alignas(16) uint32_t hist[kThetaBins];
  __shared__ uint32_t red[2][32];
  __shared__ uint32_t small[sel::kSmallList];
  __shared__ uint32_t small_n;
  __shared__ uint32_t found[3];
  __shared__ int warp_tot[32];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int h = blockIdx.x % s.Hq;
  const int seg = blockIdx.x / s.Hq;              // layer * n_seqs + seq
  const int layer = seg / s.n_seqs, seq = seg - layer * s.n_seqs;
  const int t0 = __ldg(s.cu_seqlens + seq);
  const int L = __ldg(s.cu_seqlens + seq + 1) - t0;
  const int keep = __ldg(sig_keep + seg);
  float* out = theta + (size_t)seg * s.Hq + h;
  if (keep <= 0 || keep >= L) {
    if (tid == 0) *out = keep <= 0 ? __int_as_float(0x7F800000) : __int_as_float(0xFF800000);
    return;
  }
  const float* row = scores + ((size_t)layer * s.Hq + h) * s.T + t0;

  uint32_t key[kItems];
  uint32_t lo = 0xFFFFFFFFu, hi = 0u;
#pragma unroll
  for (int j = 0; j < kItems; ++j) {
    const int i = j * kT + tid;
    key[j] = i < L ? order_key(__ldg(row + i)) : 0u;
  }
#pragma unroll
  for (int j = 0; j < kItems; ++j)
    if (j * kT + tid < L) { lo = min(lo, key[j]); hi = max(hi, key[j]); }
  lo = __reduce_min_sync(sel::kFull, lo);
  hi = __reduce_max_sync(sel::kFull, hi);
  if (lane == 0) { red[0][warp] = lo; red[1][warp] = hi; }
  for (int i = tid; i < kThetaBins; i += kT) hist[i] = 0;
  if (tid == 0) small_n = 0;
  __syncthreads();
  lo = __reduce_min_sync(sel::kFull, lane < kT / 32 ? red[0][lane] : 0xFFFFFFFFu);
  hi = __reduce_max_sync(sel::kFull, lane < kT / 32 ? red[1][lane] : 0u);
  const uint32_t base = lo, range = hi - lo;
  // From here on key[j] holds x = key - base; slots past the end of the row hold 0, the row's minimum: they add to
  // the count of the lowest values only, which a rank counted from the top (keep < L) never reaches beyond the
  // real minimum itself.
#pragma unroll
  for (int j = 0; j < kItems; ++j) key[j] = j * kT + tid < L ? key[j] - base : 0u;

  // x has `rem` significant bits; `top` is the value of the bits of x above them chosen so far
  int rem = range ? 32 - __clz(range) : 0;
  uint32_t top = 0, k_rem = (uint32_t)keep;
  bool first = true;
  while (rem > 0) {
    const int w = rem < kThetaBits ? rem : kThetaBits, shift = rem - w, n_bins = 1 << w;
    if (first) {                                             // every x counts and has no bits above the digit
#pragma unroll
      for (int j = 0; j < kItems; ++j) atomicAdd(&hist[key[j] >> shift], 1u);
    } else {
      for (int i = tid; i < n_bins; i += kT) hist[i] = 0;
      if (tid == 0) small_n = 0;
      __syncthreads();
#pragma unroll
      for (int j = 0; j < kItems; ++j)
        if (((key[j] >> 1) >> (rem - 1)) == top) atomicAdd(&hist[(key[j] >> shift) & (uint32_t)(n_bins - 1)], 1u);
    }
    first = false;
    __syncthreads();
    sel::find_digit_desc<kT>(hist, n_bins, k_rem, warp_tot, found);
    top = (top << w) | found[0];
    k_rem = found[1];
    const uint32_t live = found[2];
    rem = shift;
    if (rem > 0 && live <= (uint32_t)sel::kSmallList) {     // few candidates: one warp ranks them and finishes
#pragma unroll
      for (int j = 0; j < kItems; ++j)
        if ((key[j] >> rem) == top) small[atomicAdd(&small_n, 1u)] = key[j];
      __syncthreads();
      if (warp == 0) {
        const uint32_t x = sel::warp_rank_select32(lane < (int)live ? small[lane] : 0u, (int)live, k_rem, lane);
        if (lane == 0) *out = key_to_float(base + x);
      }
      return;
    }
    __syncthreads();                                         // hist and found are rewritten by the next step
  }
  if (tid == 0) *out = key_to_float(base + top);
}

__global__ void __launch_bounds__(kSelectThreads)
theta_stream_kernel(Shape s, const float* __restrict__ scores, const int32_t* __restrict__ sig_keep,
                    float* __restrict__ theta, int stage_row) {
  extern __shared__ uint32_t row_keys[];          // the row's order keys when it fits (stage_row), else unused
  __shared__ uint32_t hist[256];
  __shared__ uint32_t sel_prefix, sel_k;

  const int h = blockIdx.x % s.Hq;
  const int seg = blockIdx.x / s.Hq;              // layer * n_seqs + seq
  const int layer = seg / s.n_seqs, seq = seg - layer * s.n_seqs;
  const int t0 = __ldg(s.cu_seqlens + seq);
  const int L = __ldg(s.cu_seqlens + seq + 1) - t0;
  const int keep = __ldg(sig_keep + seg);
  float* out = theta + (size_t)seg * s.Hq + h;
  if (keep <= 0 || keep >= L) {
    if (threadIdx.x == 0) *out = keep <= 0 ? __int_as_float(0x7F800000) : __int_as_float(0xFF800000);
    return;
  }
  const float* row = scores + ((size_t)layer * s.Hq + h) * s.T + t0;
  const int lane = threadIdx.x & 31;

  // When the row fits, its order keys are first copied into shared memory with independent, coalesced loads
  // (the sweeps below interleave every load with warp votes and atomics, which would expose the full global
  // latency once per element).
  if (stage_row) {
#pragma unroll 4
    for (int i = threadIdx.x; i < L; i += kSelectThreads) row_keys[i] = order_key(__ldg(row + i));
    __syncthreads();
  }

  uint32_t prefix = 0;       // selected high digits so far
  uint32_t k_rem = keep;     // rank among the elements that share the prefix
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = threadIdx.x; i < 256; i += kSelectThreads) hist[i] = 0;
    __syncthreads();
    const uint32_t hi_mask = shift == 24 ? 0u : (0xFFFFFFFFu << (shift + 8));
    for (int base = 0; base < L; base += kSelectThreads) {
      const int i = base + threadIdx.x;
      const bool in = i < L;
      const uint32_t key = !in ? 0u : stage_row ? row_keys[i] : order_key(__ldg(row + i));
      const bool live = in && ((key & hi_mask) == prefix);
      const uint32_t digit = (key >> shift) & 0xFFu;
      // high digits (sign, exponent) are the same for almost every score: one add per warp then;
      // low digits are spread over the 256 bins, where plain shared-memory atomics do not collide much
      const unsigned voters = __ballot_sync(0xFFFFFFFFu, live);
      if (voters) {
        const uint32_t d0 = __shfl_sync(0xFFFFFFFFu, digit, __ffs(voters) - 1);
        if (__all_sync(0xFFFFFFFFu, !live || digit == d0)) {
          if (lane == 0) atomicAdd(&hist[d0], __popc(voters));
        } else if (live) {
          atomicAdd(&hist[digit], 1u);
        }
      }
    }
    __syncthreads();
    if (threadIdx.x < 32) {
      // lane l owns the 8 bins 255-8l .. 248-8l (descending order of value)
      uint32_t local = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) local += hist[255 - 8 * lane - j];
      uint32_t incl = local;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += v;
      }
      const uint32_t excl = incl - local;
      if (excl < k_rem && k_rem <= incl) {
        uint32_t acc = excl;
        for (int j = 0; j < 8; ++j) {
          const uint32_t c = hist[255 - 8 * lane - j];
          if (k_rem <= acc + c) {
            sel_prefix = prefix | ((uint32_t)(255 - 8 * lane - j) << shift);
            sel_k = k_rem - acc;
            break;
          }
          acc += c;
        }
      }
    }
    __syncthreads();
    prefix = sel_prefix;
    k_rem = sel_k;
    __syncthreads();
  }
  if (threadIdx.x == 0) *out = key_to_float(prefix);
}

// kImportance: also write I(t) = sum of the token's per-head scores (float64; heads ascending inside each KV
// group, then the group sums ascending: sequential IEEE additions, so the value is bit-reproducible).
// Grid: (token blocks, layers); a block owns kPackTok consecutive tokens of one layer.  Its [heads][tokens] tile of
// scores goes through shared memory: the loads are 16-byte, row-contiguous and all in flight at once (eight per
// thread at 32 heads), and the per-token walk over the heads afterwards reads shared memory without conflicts.
// The thresholds of the block's sequence sit in shared memory when all its tokens belong to one sequence (always,
// with one sequence per batch); else every thread reads its own sequence's row.
constexpr int kPackTok = 128;
#ifndef KVC_PACK_MINB
#define KVC_PACK_MINB 8                 // resident blocks per SM the pack kernel is compiled for (registers per thread)
#endif

template <bool kImportance>
__global__ void __launch_bounds__(kPackTok, KVC_PACK_MINB)
signature_pack_kernel(Shape s, const float* __restrict__ scores, const float* __restrict__ theta,
                      uint32_t* __restrict__ sigs, double* __restrict__ importance, int vec_ok) {
  extern __shared__ float4 tile4[];                   // [Hq][kPackTok] float
  float* tile = reinterpret_cast<float*>(tile4);
  __shared__ float th_sh[128];
  const int layer = blockIdx.y;
  const int tok0 = blockIdx.x * kPackTok, tok = tok0 + threadIdx.x;
  const int n_tok = min(kPackTok, s.T - tok0);
  const float* base = scores + (size_t)layer * s.Hq * s.T + tok0;
  if (vec_ok && n_tok == kPackTok) {                  // rows start on 16-byte boundaries
#pragma unroll 8
    for (int i = threadIdx.x; i < s.Hq * (kPackTok / 4); i += kPackTok) {
      const int h = i / (kPackTok / 4), c = i % (kPackTok / 4);
      tile4[i] = __ldg(reinterpret_cast<const float4*>(base + (size_t)h * s.T) + c);
    }
  } else {
#pragma unroll 8
    for (int h = 0; h < s.Hq; ++h)
      tile[h * kPackTok + threadIdx.x] = (int)threadIdx.x < n_tok ? __ldg(base + (size_t)h * s.T + threadIdx.x) : 0.f;
  }
  const int seq0 = seq_of_token(s.cu_seqlens, s.n_seqs, tok0);
  const bool one_seq = tok0 + n_tok <= __ldg(s.cu_seqlens + seq0 + 1);
  if (one_seq)
    for (int h = threadIdx.x; h < s.Hq; h += kPackTok) th_sh[h] = __ldg(theta + ((size_t)layer * s.n_seqs + seq0) * s.Hq + h);
  __syncthreads();
  if ((int)threadIdx.x >= n_tok) return;
  const float* th = one_seq ? th_sh
                            : theta + ((size_t)layer * s.n_seqs + seq_of_token(s.cu_seqlens, s.n_seqs, tok)) * s.Hq;
  const float* col = tile + threadIdx.x;
  uint32_t* out = sigs + ((size_t)layer * s.T + tok) * s.W;
  double total = 0.0, group = 0.0;
  int in_group = 0;
  for (int w = 0; w < s.W; ++w) {
    uint32_t word = 0;
    const int nb = min(32, s.Hq - 32 * w);
#pragma unroll 8
    for (int b = 0; b < nb; ++b) {
      const float v = col[(32 * w + b) * kPackTok];
      word |= (uint32_t)(v >= th[32 * w + b]) << b;
      if constexpr (kImportance) {
        group = __dadd_rn(group, (double)v);
        if (++in_group == s.G) { total = __dadd_rn(total, group); group = 0.0; in_group = 0; }
      }
    }
    out[w] = word;
  }
  if constexpr (kImportance) importance[(size_t)layer * s.T + tok] = __dadd_rn(total, 0.0);       // -0.0 -> +0.0
}

template <int kT, int kItems, int kMinB>
void launch_theta(const Shape& s, const float* scores, const int32_t* sig_keep, float* theta, unsigned blocks,
                  cudaStream_t stream) {
  theta_select_kernel<kT, kItems, kMinB><<<blocks, kT, 0, stream>>>(s, scores, sig_keep, theta);
}

}  // namespace

int launch_signature(const Shape& s, const float* scores, const int32_t* sig_keep, const float* theta_in,
                     uint32_t* sigs, float* theta, double* importance, cudaStream_t stream) {
  if (s.T == 0) return KVCRUSH_OK;
  const float* th = theta_in;
  if (!theta_in) {
    const unsigned blocks = (unsigned)s.n_layers * s.n_seqs * s.Hq;
    const int m = s.max_seqlen;
    if (m <= 2048) launch_theta<256, 8, 8>(s, scores, sig_keep, theta, blocks, stream);
    else if (m <= 4096) launch_theta<512, 8, 4>(s, scores, sig_keep, theta, blocks, stream);
    else if (m <= 8192) launch_theta<512, 16, 4>(s, scores, sig_keep, theta, blocks, stream);
    else if (m <= 16384) launch_theta<512, 32, 1>(s, scores, sig_keep, theta, blocks, stream);
    else if (m <= 32768) launch_theta<1024, 32, 1>(s, scores, sig_keep, theta, blocks, stream);
    else {
      const size_t row_bytes = (size_t)m * sizeof(uint32_t);
      const int stage_row = row_bytes <= 200 * 1024;
      const size_t dyn = stage_row ? row_bytes : 0;
      if (dyn > 40 * 1024 &&
          cudaFuncSetAttribute(theta_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
        return KVCRUSH_ERR_CUDA;
      theta_stream_kernel<<<blocks, kSelectThreads, dyn, stream>>>(s, scores, sig_keep, theta, stage_row);
    }
    if (check_launch() != KVCRUSH_OK) return KVCRUSH_ERR_CUDA;
    th = theta;
  }
  const dim3 grid((unsigned)((s.T + kPackTok - 1) / kPackTok), (unsigned)s.n_layers);
  const size_t dyn = (size_t)s.Hq * kPackTok * sizeof(float);
  // 16-byte loads need every (layer, head) row to start on a 16-byte boundary
  const int vec_ok = s.T % 4 == 0 && reinterpret_cast<uintptr_t>(scores) % 16 == 0;
  if (importance) {
    if (dyn > 48 * 1024 && cudaFuncSetAttribute(signature_pack_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
      return KVCRUSH_ERR_CUDA;
    signature_pack_kernel<true><<<grid, kPackTok, dyn, stream>>>(s, scores, th, sigs, importance, vec_ok);
  } else {
    if (dyn > 48 * 1024 && cudaFuncSetAttribute(signature_pack_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
      return KVCRUSH_ERR_CUDA;
    signature_pack_kernel<false><<<grid, kPackTok, dyn, stream>>>(s, scores, th, sigs, nullptr, vec_ok);
  }
  return check_launch();
}

// ---------------------------------------------------------------------------------------------------
// kvcrush_signature_static: the same two kernels, thresholds kept in library-owned device memory.
// ---------------------------------------------------------------------------------------------------
namespace {

// Thresholds of one call, [n_layers][n_seqs][n_q_heads].  Lives in the library image on every device.
static __device__ __align__(256) float g_static_theta[KVCRUSH_STATIC_THETA_MAX];

constexpr int kMaxDevices = 64;

// Device address of g_static_theta on the current device.  In host code the symbol's name is only a
// handle; the address a kernel can use comes from cudaGetSymbolAddress, looked up once per device.
int static_theta_ptr(float** out) {
  static float* cached[kMaxDevices] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return KVCRUSH_ERR_CUDA;
  float* p = __atomic_load_n(&cached[dev], __ATOMIC_ACQUIRE);
  if (!p) {
    void* addr = nullptr;
    if (cudaGetSymbolAddress(&addr, g_static_theta) != cudaSuccess || !addr) return KVCRUSH_ERR_CUDA;
    p = static_cast<float*>(addr);
    __atomic_store_n(&cached[dev], p, __ATOMIC_RELEASE);
  }
  *out = p;
  return KVCRUSH_OK;
}

}  // namespace
}  // namespace kvc

extern "C" int kvcrush_signature_static(const kvcrush_problem_t* problem, const float* scores_dev,
                                        const int32_t* sig_keep_dev, uint32_t* sigs_dev,
                                        int32_t* status_dev, void* stream) {
  kvc::Shape s;
  const int rc = kvc::shape_from_problem(problem, &s);
  if (rc != KVCRUSH_OK) return rc;
  if (!scores_dev || !sig_keep_dev || !sigs_dev || !status_dev) return KVCRUSH_ERR_INVALID_ARG;
  if ((long long)s.n_layers * s.n_seqs * s.Hq > KVCRUSH_STATIC_THETA_MAX) return KVCRUSH_ERR_STATIC_LIMIT;
  float* theta = nullptr;
  const int prc = kvc::static_theta_ptr(&theta);
  if (prc != KVCRUSH_OK) return prc;
  return kvc::launch_signature(s, scores_dev, sig_keep_dev, nullptr, sigs_dev, theta, nullptr,
                               static_cast<cudaStream_t>(stream));
}
