// Stage 2: per-head thresholds and packed binary signatures (Algorithm 1 and Sec. 3.1 of the paper).
//
//   theta_select_kernel   theta = keep-th largest score of one (layer, sequence, head): an exact
//                         MSB-first radix select over order-preserving 32-bit keys (4 sweeps of 8
//                         bits, shared-memory histograms with a one-add-per-warp path for uniform digits).
//   binarise_pack_kernel  one thread per (layer, token): compares the token's score of every head
//                         with that head's threshold and packs the bits.  Lanes are consecutive
//                         tokens, so every per-head load is a coalesced 128-byte row.
#include "common.cuh"

namespace kvc {

namespace {

constexpr int kSelectThreads = 512;

// float -> uint32 such that a < b  <=>  key(a) < key(b) (for non-NaN values)
__device__ __forceinline__ uint32_t order_key(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_to_float(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

__global__ void __launch_bounds__(kSelectThreads)
theta_select_kernel(Shape s, const float* __restrict__ scores, const int32_t* __restrict__ sig_keep,
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

__global__ void __launch_bounds__(256)
binarise_pack_kernel(Shape s, const float* __restrict__ scores, const float* __restrict__ theta,
                     uint32_t* __restrict__ sigs) {
  const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= (long long)s.n_layers * s.T) return;
  const int layer = (int)(gid / s.T), tok = (int)(gid - (long long)layer * s.T);
  const int seq = seq_of_token(s.cu_seqlens, s.n_seqs, tok);
  const float* sc = scores + (size_t)layer * s.Hq * s.T + tok;
  const float* th = theta + ((size_t)layer * s.n_seqs + seq) * s.Hq;
  uint32_t* out = sigs + ((size_t)layer * s.T + tok) * s.W;
  for (int w = 0; w < s.W; ++w) {
    uint32_t word = 0;
    const int h_end = min(32, s.Hq - 32 * w);
    for (int b = 0; b < h_end; ++b) {
      const int h = 32 * w + b;
      word |= (uint32_t)(__ldg(sc + (size_t)h * s.T) >= __ldg(th + h)) << b;
    }
    out[w] = word;
  }
}

}  // namespace

int launch_signature(const Shape& s, const float* scores, const int32_t* sig_keep, const float* theta_in,
                     uint32_t* sigs, float* theta, cudaStream_t stream) {
  if (s.T == 0) return KVCRUSH_OK;
  const float* th = theta_in;
  if (!theta_in) {
    const unsigned blocks = (unsigned)s.n_layers * s.n_seqs * s.Hq;
    const size_t row_bytes = (size_t)s.max_seqlen * sizeof(uint32_t);
    const int stage_row = row_bytes <= 96 * 1024;
    const size_t dyn = stage_row ? row_bytes : 0;
    if (dyn > 40 * 1024 &&
        cudaFuncSetAttribute(theta_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
      return KVCRUSH_ERR_CUDA;
    theta_select_kernel<<<blocks, kSelectThreads, dyn, stream>>>(s, scores, sig_keep, theta, stage_row);
    if (check_launch() != KVCRUSH_OK) return KVCRUSH_ERR_CUDA;
    th = theta;
  }
  const long long n = (long long)s.n_layers * s.T;
  binarise_pack_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(s, scores, th, sigs);
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
  return kvc::launch_signature(s, scores_dev, sig_keep_dev, nullptr, sigs_dev, theta,
                               static_cast<cudaStream_t>(stream));
}
