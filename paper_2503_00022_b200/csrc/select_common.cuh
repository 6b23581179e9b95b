// Block-wide building blocks shared by the token-level and the page-level selection kernels:
// exact top-k marking of 64-bit keys and emission of the kept set from two membership masks.
#pragma once

#include "common.cuh"

namespace kvc {
namespace sel {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr unsigned kFull = 0xFFFFFFFFu;

struct Scratch {
  uint32_t hist[256];
  unsigned long long sel_prefix;
  uint32_t sel_k;
  int warp_tot[kWarps];
};

__device__ __forceinline__ uint32_t head_mask(int Hq, int w) {
  const int n = Hq - 32 * w;
  return n >= 32 ? 0xFFFFFFFFu : ((1u << n) - 1u);
}

// Contiguous item range of a warp: a multiple of 32 items, so that mask words do not straddle warps.
__device__ __forceinline__ void warp_range(int n, int warp, int& r_lo, int& r_hi) {
  const int n_words = (n + 31) >> 5;
  const int per_warp = ((n_words + kWarps - 1) / kWarps) * 32;
  r_lo = min(n, warp * per_warp);
  r_hi = min(n, r_lo + per_warp);
}

// Sets bit i of imp_mask for the k items with the largest keys[0..n); equal keys are admitted in ascending
// index order.  Exact MSB-first radix select (8 digits of 8 bits), then one ordered pass.  Called by all
// threads of the block; imp_mask must be zero on entry; 0 < k < n.
__device__ __forceinline__ void mark_top_keys(const unsigned long long* keys, int n, int k, uint32_t* imp_mask,
                                              Scratch& sc) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned lt_mask = (1u << lane) - 1u;
  int r_lo, r_hi;
  warp_range(n, warp, r_lo, r_hi);
  unsigned long long prefix = 0;
  uint32_t k_rem = k;
  for (int shift = 56; shift >= 0; shift -= 8) {
    for (int i = tid; i < 256; i += kThreads) sc.hist[i] = 0;
    __syncthreads();
    const unsigned long long hi_mask = shift == 56 ? 0ull : (~0ull << (shift + 8));
    for (int base = 0; base < n; base += kThreads) {
      const int i = base + tid;
      const bool in = i < n;
      const unsigned long long key = in ? keys[i] : 0ull;
      const bool live = in && ((key & hi_mask) == prefix);
      const uint32_t digit = (uint32_t)(key >> shift) & 0xFFu;
      // high digits (sign, exponent) are the same for almost every key: one add per warp then;
      // low digits are spread over the 256 bins, where plain shared-memory atomics do not collide much
      const unsigned voters = __ballot_sync(kFull, live);
      if (voters) {
        const uint32_t d0 = __shfl_sync(kFull, digit, __ffs(voters) - 1);
        if (__all_sync(kFull, !live || digit == d0)) {
          if (lane == 0) atomicAdd(&sc.hist[d0], __popc(voters));
        } else if (live) {
          atomicAdd(&sc.hist[digit], 1u);
        }
      }
    }
    __syncthreads();
    if (warp == 0) {
      uint32_t local = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) local += sc.hist[255 - 8 * lane - j];
      uint32_t incl = local;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_up_sync(kFull, incl, d);
        if (lane >= d) incl += v;
      }
      const uint32_t excl = incl - local;
      if (excl < k_rem && k_rem <= incl) {
        uint32_t acc = excl;
        for (int j = 0; j < 8; ++j) {
          const uint32_t c = sc.hist[255 - 8 * lane - j];
          if (k_rem <= acc + c) {
            sc.sel_prefix = prefix | ((unsigned long long)(255 - 8 * lane - j) << shift);
            sc.sel_k = k_rem - acc;
            break;
          }
          acc += c;
        }
      }
    }
    __syncthreads();
    prefix = sc.sel_prefix;
    k_rem = sc.sel_k;
    __syncthreads();
  }
  // prefix = the k-th largest key; k_rem = how many keys equal to it are admitted
  const unsigned long long kth = prefix;
  int n_eq = 0;
  for (int i = r_lo + lane; i < r_hi; i += 32) n_eq += (keys[i] == kth);
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) n_eq += __shfl_xor_sync(kFull, n_eq, d);
  if (lane == 0) sc.warp_tot[warp] = n_eq;
  __syncthreads();
  int eq_before = 0;
  for (int w = 0; w < warp; ++w) eq_before += sc.warp_tot[w];
  for (int base = r_lo; base < r_hi; base += 32) {
    const int i = base + lane;
    const unsigned long long key = i < r_hi ? keys[i] : 0ull;
    const bool eq = i < r_hi && key == kth;
    const unsigned eq_b = __ballot_sync(kFull, eq);
    const bool imp = i < r_hi && (key > kth || (eq && (uint32_t)(eq_before + __popc(eq_b & lt_mask)) < k_rem));
    const unsigned imp_b = __ballot_sync(kFull, imp);
    if (lane == 0) imp_mask[base >> 5] = imp_b;
    eq_before += __popc(eq_b);
  }
  __syncthreads();
}

// Writes the members of imp_mask | rep_mask in ascending order (kind: 1 for members of rep_mask).
// Called by all threads of the block after the masks are complete.
__device__ __forceinline__ void emit_kept(const uint32_t* imp_mask, const uint32_t* rep_mask, int n_words,
                                          int32_t* out_idx, uint8_t* out_kind, Scratch& sc) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wpt = (n_words + kThreads - 1) / kThreads;      // mask words per thread, contiguous
  const int w_lo = min(n_words, tid * wpt), w_hi = min(n_words, w_lo + wpt);
  int cnt = 0;
  for (int w = w_lo; w < w_hi; ++w) cnt += __popc(imp_mask[w] | rep_mask[w]);
  int incl = cnt;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int v = __shfl_up_sync(kFull, incl, d);
    if (lane >= d) incl += v;
  }
  __syncthreads();                          // warp_tot may still be read by an earlier phase
  if (lane == 31) sc.warp_tot[warp] = incl;
  __syncthreads();
  int pos = incl - cnt;
  for (int w = 0; w < warp; ++w) pos += sc.warp_tot[w];
  for (int w = w_lo; w < w_hi; ++w) {
    const uint32_t rep = rep_mask[w];
    uint32_t bits = imp_mask[w] | rep;
    while (bits) {
      const int b = __ffs(bits) - 1;
      bits &= bits - 1;
      out_idx[pos] = 32 * w + b;
      if (out_kind) out_kind[pos] = (rep >> b) & 1u;
      ++pos;
    }
  }
}

}  // namespace sel
}  // namespace kvc
