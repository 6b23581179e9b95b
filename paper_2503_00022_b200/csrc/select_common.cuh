// Block-wide building blocks shared by the signature, the token-level and the page-level selection kernels:
// the search for the k-th largest key by radix histograms, exact top-k marking of 64-bit keys and emission of
// the kept set from two membership masks.
#pragma once

#include "common.cuh"

namespace kvc {
namespace sel {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kDigitBits = 11;                 // radix digit of the 64-bit selection
constexpr int kBins = 1 << kDigitBits;
constexpr int kSmallList = 32;                 // candidates one warp ranks directly

struct Scratch {
  alignas(16) uint32_t hist[kBins];
  unsigned long long red[2][kWarps];           // per-warp minimum / maximum
  unsigned long long small[kSmallList];
  unsigned long long sel_x;                    // result of a search step
  uint32_t sel[3];                             // digit, remaining rank, live keys
  uint32_t small_n;
  int warp_tot[kWarps];
};

__device__ __forceinline__ uint32_t head_mask(int Hq, int w) {
  const int n = Hq - 32 * w;
  return n >= 32 ? 0xFFFFFFFFu : ((1u << n) - 1u);
}

// Sum of tot[0 .. warp) for every thread of warp `warp`: one load per lane and a warp reduction instead of a serial
// walk (the last warp would otherwise do 31 dependent loads).  n_warps <= 32.
__device__ __forceinline__ int warps_before(const int* tot, int warp, int lane) {
  return __reduce_add_sync(kFull, lane < warp ? tot[lane] : 0);
}

// Contiguous item range of a warp: a multiple of 32 items, so that mask words do not straddle warps.
__device__ __forceinline__ void warp_range(int n, int warp, int& r_lo, int& r_hi) {
  const int n_words = (n + 31) >> 5;
  const int per_warp = ((n_words + kWarps - 1) / kWarps) * 32;
  r_lo = min(n, warp * per_warp);
  r_hi = min(n, r_lo + per_warp);
}

// The digit that holds the k_rem-th largest key, from a complete histogram of one digit position (bins in
// ascending digit order, counted from the top): out[0] = digit, out[1] = rank left inside that digit's bin,
// out[2] = keys in the bin.  Called by all kT threads of the block; k_rem is at most the histogram's total.
// The histogram must be complete (a barrier lies between its last update and this call); the result is
// visible to every thread on return.
template <int kT>
__device__ __forceinline__ void find_digit_desc(const uint32_t* hist, int n_bins, uint32_t k_rem, int* warp_tot,
                                                uint32_t* out) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per = n_bins >= kT ? n_bins / kT : 1;           // bins per thread, walked from the top digit down
  const int n_act = n_bins / per;
  uint32_t local = 0;
  if (tid < n_act) {
    const int first = n_bins - (tid + 1) * per;              // the thread's bins are [first, first + per)
    if (per % 4 == 0) {                                      // 16-byte loads: consecutive threads, consecutive quads
      const uint4* q = reinterpret_cast<const uint4*>(hist + first);
      for (int j = 0; j < per / 4; ++j) { const uint4 v = q[j]; local += (v.x + v.y) + (v.z + v.w); }
    } else {
      for (int j = 0; j < per; ++j) local += hist[first + j];
    }
  }
  uint32_t incl = local;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t v = __shfl_up_sync(kFull, incl, d);
    if (lane >= d) incl += v;
  }
  if (lane == 31) warp_tot[warp] = (int)incl;
  __syncthreads();
  uint32_t excl = incl - local;
  excl += (uint32_t)warps_before(warp_tot, warp, lane);
  if (tid < n_act && excl < k_rem && k_rem <= excl + local) {
    uint32_t acc = excl;
    for (int j = 0; j < per; ++j) {
      const int bin = n_bins - 1 - (tid * per + j);
      const uint32_t c = hist[bin];
      if (k_rem <= acc + c) {
        out[0] = (uint32_t)bin; out[1] = k_rem - acc; out[2] = c;
        break;
      }
      acc += c;
    }
  }
  __syncthreads();
}

// One warp ranks at most 32 candidates held one per lane (lanes >= n hold nothing): returns in every lane the
// k_rem-th largest value, sets k_out to the rank left among the candidates equal to it and n_equal to their number.
__device__ __forceinline__ unsigned long long warp_rank_select(unsigned long long v, int n, uint32_t k_rem, int lane,
                                                               uint32_t& k_out, uint32_t& n_equal) {
  uint32_t gt = 0, ge = 0;
  for (int j = 0; j < n; ++j) {
    const unsigned long long o = __shfl_sync(kFull, v, j);
    gt += o > v;
    ge += o >= v;
  }
  const bool hit = lane < n && gt < k_rem && k_rem <= ge;
  const unsigned who = __ballot_sync(kFull, hit);
  const int src = __ffs(who) - 1;                     // equal candidates all qualify: any of them
  const uint32_t gt_src = __shfl_sync(kFull, gt, src);
  k_out = k_rem - gt_src;
  n_equal = __shfl_sync(kFull, ge, src) - gt_src;
  return __shfl_sync(kFull, v, src);
}

// The same for 32-bit candidates (one shuffle per candidate instead of two).
__device__ __forceinline__ uint32_t warp_rank_select32(uint32_t v, int n, uint32_t k_rem, int lane) {
  uint32_t gt = 0, ge = 0;
  for (int j = 0; j < n; ++j) {
    const uint32_t o = __shfl_sync(kFull, v, j);
    gt += o > v;
    ge += o >= v;
  }
  const bool hit = lane < n && gt < k_rem && k_rem <= ge;
  const unsigned who = __ballot_sync(kFull, hit);
  return __shfl_sync(kFull, v, __ffs(who) - 1);
}

// Sets bit i of imp_mask for the k items with the largest keys[0..n); equal keys are admitted in ascending
// index order.  Exact: the k-th largest key is found by radix histograms over (key - smallest key), starting at
// the top bit in which the keys of this segment differ at all - the digits are then spread over the bins whatever
// the keys' common magnitude -, and as soon as at most 32 candidates are left one warp ranks them directly; then
// one ordered pass marks the members.  Called by all threads of the block; imp_mask must be zero on entry;
// 0 < k < n.
__device__ __forceinline__ void mark_top_keys(const unsigned long long* keys, int n, int k, uint32_t* imp_mask,
                                              Scratch& sc) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned lt_mask = (1u << lane) - 1u;
  int r_lo, r_hi;
  warp_range(n, warp, r_lo, r_hi);

  // smallest and largest key
  unsigned long long lo = ~0ull, hi = 0ull;
  for (int i = tid; i < n; i += kThreads) {
    const unsigned long long key = keys[i];
    lo = key < lo ? key : lo;
    hi = key > hi ? key : hi;
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    const unsigned long long a = __shfl_xor_sync(kFull, lo, d), b = __shfl_xor_sync(kFull, hi, d);
    lo = a < lo ? a : lo;
    hi = b > hi ? b : hi;
  }
  if (lane == 0) { sc.red[0][warp] = lo; sc.red[1][warp] = hi; }
  __syncthreads();
  lo = sc.red[0][lane];
  hi = sc.red[1][lane];
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    const unsigned long long a = __shfl_xor_sync(kFull, lo, d), b = __shfl_xor_sync(kFull, hi, d);
    lo = a < lo ? a : lo;
    hi = b > hi ? b : hi;
  }
  const unsigned long long base = lo, range = hi - lo;

  // x = key - base has `rem` significant bits; `top` is the value of the bits of x above them chosen so far
  int rem = range ? 64 - __clzll((long long)range) : 0;
  unsigned long long top = 0;
  uint32_t k_rem = (uint32_t)k;
  uint32_t n_equal = (uint32_t)n;                      // keys equal to the k-th largest (all of them when range == 0)
  bool first = true;
  while (rem > 0) {
    const int w = rem < kDigitBits ? rem : kDigitBits, shift = rem - w, n_bins = 1 << w;
    for (int i = tid; i < n_bins; i += kThreads) sc.hist[i] = 0;
    if (tid == 0) sc.small_n = 0;
    __syncthreads();
    if (first) {                                       // every key counts and has no bits above the digit
      for (int i = tid; i < n; i += kThreads) atomicAdd(&sc.hist[(uint32_t)((keys[i] - base) >> shift)], 1u);
    } else {
      for (int i = tid; i < n; i += kThreads) {
        const unsigned long long x = keys[i] - base;
        if (((x >> 1) >> (rem - 1)) == top) atomicAdd(&sc.hist[(uint32_t)(x >> shift) & (uint32_t)(n_bins - 1)], 1u);
      }
    }
    first = false;
    __syncthreads();
    find_digit_desc<kThreads>(sc.hist, n_bins, k_rem, sc.warp_tot, sc.sel);
    top = (top << w) | sc.sel[0];
    k_rem = sc.sel[1];
    const uint32_t live = sc.sel[2];
    n_equal = live;                                    // exact once no bits are left
    rem = shift;
    if (rem > 0 && live <= (uint32_t)kSmallList) {     // few candidates: one warp ranks their remaining bits
      for (int i = tid; i < n; i += kThreads) {
        const unsigned long long x = keys[i] - base;
        if ((x >> rem) == top) sc.small[atomicAdd(&sc.small_n, 1u)] = x;
      }
      __syncthreads();
      if (warp == 0) {
        uint32_t k_out, n_eq_out;
        const unsigned long long v = warp_rank_select(lane < (int)live ? sc.small[lane] : 0ull, (int)live, k_rem, lane, k_out, n_eq_out);
        if (lane == 0) { sc.sel_x = v; sc.sel[1] = k_out; sc.sel[2] = n_eq_out; }
      }
      __syncthreads();
      top = sc.sel_x;
      k_rem = sc.sel[1];
      n_equal = sc.sel[2];
      rem = 0;
    }
    __syncthreads();                                   // sc.sel and sc.hist are rewritten by the next step
  }
  // kth = the k-th largest key; k_rem of the n_equal keys equal to it are admitted, in ascending index order
  const unsigned long long kth = base + top;
  if (k_rem == n_equal) {                              // no tie is cut (the usual case): everything >= kth is in
    for (int base_i = r_lo; base_i < r_hi; base_i += 32) {
      const int i = base_i + lane;
      const unsigned imp_b = __ballot_sync(kFull, i < r_hi && keys[i] >= kth);
      if (lane == 0) imp_mask[base_i >> 5] = imp_b;
    }
    __syncthreads();
    return;
  }
  int n_eq = 0;
  for (int i = r_lo + lane; i < r_hi; i += 32) n_eq += (keys[i] == kth);
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) n_eq += __shfl_xor_sync(kFull, n_eq, d);
  if (lane == 0) sc.warp_tot[warp] = n_eq;
  __syncthreads();
  int eq_before = 0;
  eq_before += warps_before(sc.warp_tot, warp, lane);
  for (int base_i = r_lo; base_i < r_hi; base_i += 32) {
    const int i = base_i + lane;
    const unsigned long long key = i < r_hi ? keys[i] : 0ull;
    const bool eq = i < r_hi && key == kth;
    const unsigned eq_b = __ballot_sync(kFull, eq);
    const bool imp = i < r_hi && (key > kth || (eq && (uint32_t)(eq_before + __popc(eq_b & lt_mask)) < k_rem));
    const unsigned imp_b = __ballot_sync(kFull, imp);
    if (lane == 0) imp_mask[base_i >> 5] = imp_b;
    eq_before += __popc(eq_b);
  }
  __syncthreads();
}

// Writes the members of imp_mask | rep_mask in ascending order (kind: 1 for members of rep_mask).
// Called by all threads of the block after the masks are complete.
__device__ __forceinline__ void emit_kept(const uint32_t* imp_mask, const uint32_t* rep_mask, int n_words,
                                          int32_t* out_idx, uint8_t* out_kind, Scratch& sc) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // every thread takes a contiguous run of mask BYTES (8 items each): with fewer words than threads a word-wise
  // split would leave most threads idle and the others with up to 32 serial stores
  const int n_bytes = 4 * n_words;
  const int bpt = (n_bytes + kThreads - 1) / kThreads;
  const int b_lo = min(n_bytes, tid * bpt), b_hi = min(n_bytes, b_lo + bpt);
  auto byte_of = [](const uint32_t* mask, int b) -> uint32_t { return (mask[b >> 2] >> (8 * (b & 3))) & 0xFFu; };
  int cnt = 0;
  for (int b = b_lo; b < b_hi; ++b) cnt += __popc(byte_of(imp_mask, b) | byte_of(rep_mask, b));
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
  pos += warps_before(sc.warp_tot, warp, lane);
  for (int b = b_lo; b < b_hi; ++b) {
    const uint32_t rep = byte_of(rep_mask, b);
    uint32_t bits = byte_of(imp_mask, b) | rep;
    while (bits) {
      const int k = __ffs(bits) - 1;
      bits &= bits - 1;
      out_idx[pos] = 8 * b + k;
      if (out_kind) out_kind[pos] = (rep >> k) & 1u;
      ++pos;
    }
  }
}

}  // namespace sel
}  // namespace kvc
