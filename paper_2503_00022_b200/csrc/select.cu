// Stage 3: the kept set of every (layer, sequence) segment (Sec. 3 and Algorithm 2 of the paper).
//
//   importance_kernel      I(t) = sum of the per-head scores of token t (H2O's cumulative attention),
//                          float64, heads added in ascending order inside each KV group and the
//                          group sums added in ascending order; stored as an order-preserving
//                          64-bit key.  One thread per (layer, token), coalesced per-head rows.
//                          Skipped when the caller hands over I(t) (the signature stage can write it
//                          from the loads it does anyway).
//   select_segment_kernel  one CTA per segment:
//                            1. exact radix select of the B_imp-th largest key, ties admitted in
//                               ascending token order                         -> important set
//                            2. anchor; d_t = popc(sig_t xor anchor) for the other tokens
//                            3. stable counting sort by (d_t, t): every warp owns a contiguous
//                               token range, per-warp histograms, one scan, ordered scatter
//                            4. equal-frequency buckets of the sorted order; per bucket the member
//                               minimising  sum_{h: bit set} (m - 2 n_h)  (= L1 distance to the
//                               per-bit mean, up to a constant), ties to the lower token
//                            5. kept = important U representatives, ascending token index
// All decisions are integer or exact float64 comparisons, so the result is unique.
#include "select_common.cuh"

namespace kvc {

namespace {

using sel::kThreads;
using sel::kWarps;
using sel::kFull;
using sel::head_mask;
constexpr int kMaxBins = 129;              // Hamming distances 0..128

// Order-preserving 64-bit key of a float64 importance; tokens kept by decree (the first keep_initial and the last
// keep_recent of a sequence of L tokens) rank as +infinity.
__device__ __forceinline__ unsigned long long importance_key(double v, int t, int L, int keep_initial, int keep_recent) {
  if (t < keep_initial || t >= L - keep_recent) v = __longlong_as_double(0x7FF0000000000000LL);
  const unsigned long long b = (unsigned long long)__double_as_longlong(v);
  return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
}

__global__ void __launch_bounds__(256)
importance_kernel(Shape s, const float* __restrict__ scores, int keep_initial, int keep_recent,
                  unsigned long long* __restrict__ keys) {
  const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= (long long)s.n_layers * s.T) return;
  const int layer = (int)(gid / s.T), tok = (int)(gid - (long long)layer * s.T);
  const float* sc = scores + (size_t)layer * s.Hq * s.T + tok;
  // the additions are sequential by definition (fixed order = bit-reproducible ranking); the loads are not,
  // so they are issued eight at a time ahead of the adds that consume them
  double total = 0.0, group = 0.0;
  int in_group = 0;
  for (int h0 = 0; h0 < s.Hq; h0 += 8) {
    float v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = h0 + j < s.Hq ? __ldg(sc + (size_t)(h0 + j) * s.T) : 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (h0 + j < s.Hq) {
        group = __dadd_rn(group, (double)v[j]);
        if (++in_group == s.G) { total = __dadd_rn(total, group); group = 0.0; in_group = 0; }
      }
    }
  }
  total = __dadd_rn(total, 0.0);           // -0.0 -> +0.0
  int t = 0, L = 0x7FFFFFFF;
  if (keep_recent > 0 || keep_initial > 0) {   // the first / last tokens of a sequence are important by decree
    const int seq = seq_of_token(s.cu_seqlens, s.n_seqs, tok);
    t = tok - __ldg(s.cu_seqlens + seq);
    L = __ldg(s.cu_seqlens + seq + 1) - __ldg(s.cu_seqlens + seq);
  }
  keys[gid] = importance_key(total, t, L, keep_initial, keep_recent);
}

// Keys from an importance array the caller supplies (segments too long for the shared-memory copy, where the
// conversion happens otherwise).
__global__ void __launch_bounds__(256)
importance_keys_kernel(Shape s, const double* __restrict__ imp, int keep_initial, int keep_recent,
                       unsigned long long* __restrict__ keys) {
  const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= (long long)s.n_layers * s.T) return;
  const int tok = (int)(gid % s.T);
  const int seq = seq_of_token(s.cu_seqlens, s.n_seqs, tok);
  const int t0 = __ldg(s.cu_seqlens + seq);
  keys[gid] = importance_key(imp[gid], tok - t0, __ldg(s.cu_seqlens + seq + 1) - t0, keep_initial, keep_recent);
}

// sum over the GW lanes of this lane's group of popc(mine & theirs); lanes without a member hold zeros
template <int W, int GW>
__device__ __forceinline__ int group_and_popc(const uint32_t (&mine)[4]) {
  int shared = 0;
#pragma unroll
  for (int u = 0; u < GW; ++u)
#pragma unroll
    for (int w = 0; w < W; ++w) shared += __popc(mine[w] & __shfl_sync(kFull, mine[w], u, GW));
  return shared;
}

struct SelectArgs {
  const unsigned long long* keys;     // [n_layers][T] importance keys; or, when NULL,
  const double* imp;                  // [n_layers][T] importance values, turned into keys while they are staged
  int keep_initial, keep_recent;      // tokens important by decree (applied with imp; keys have them built in)
  const uint32_t* sigs;               // [n_layers][T][W]
  const int32_t* budget_imp;
  const int32_t* budget_rep;
  int anchor_mode;
  const uint32_t* anchor_bits;
  int anchor_per_segment;
  const int32_t* cu_kept;
  int32_t* idx;
  uint8_t* kind;
  int32_t* n_kept;                    // optional [n_layers][n_seqs]: tokens kept per segment
  int32_t* sorted;                    // [n_layers][T] scratch: grouped tokens in (d, t) order
  int mask_words;                     // words of one membership mask in shared memory
  int stage_words;                    // max_seqlen rounded up to a multiple of 4 (one staged int32 per token)
  int stage_sorted, stage_sig, stage_keys;   // which per-segment arrays are copied into shared memory
};

template <int W>                       // signature words per token (compile time: the per-word loops unroll)
__global__ void __launch_bounds__(kThreads, 1)
select_segment_kernel(Shape s, SelectArgs a) {
  extern __shared__ uint32_t dyn_smem[];
  uint32_t* imp_mask = dyn_smem;
  uint32_t* rep_mask = dyn_smem + a.mask_words;

  __shared__ sel::Scratch sc;
  __shared__ int warp_hist[kWarps][kMaxBins];
  __shared__ int bin_base[kMaxBins + 1];
  __shared__ int bit_cnt[128];
  __shared__ uint32_t anchor_sh[4];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned lt_mask = (1u << lane) - 1u;
  const int seg = blockIdx.x;
  const int layer = seg / s.n_seqs, seq = seg - layer * s.n_seqs;
  const int t0 = __ldg(s.cu_seqlens + seq);
  const int L = __ldg(s.cu_seqlens + seq + 1) - t0;
  const int b_imp = max(0, __ldg(a.budget_imp + seg));
  const int b_rep = max(0, __ldg(a.budget_rep + seg));
  int32_t* out_idx = a.idx + __ldg(a.cu_kept + seg);
  uint8_t* out_kind = a.kind ? a.kind + __ldg(a.cu_kept + seg) : nullptr;

  if (a.n_kept && tid == 0) a.n_kept[seg] = (int)min((long long)b_imp + b_rep, (long long)L);
  if ((long long)b_imp + b_rep >= L) {             // budget covers the sequence: keep everything
    for (int i = tid; i < L; i += kThreads) {
      out_idx[i] = i;
      if (out_kind) out_kind[i] = 0;
    }
    return;
  }

  // The segment's arrays are read many times with dependent addresses (8 radix sweeps, two counting-sort
  // sweeps, one gather per bucket), so whatever fits is first copied into shared memory; the rest is read
  // through L2.  The pointers below are generic and point to either place.
  const unsigned long long* keys = a.keys ? a.keys + (size_t)layer * s.T + t0 : nullptr;
  const uint32_t* sig = a.sigs + ((size_t)layer * s.T + t0) * W;
  int32_t* sorted = a.sorted + (size_t)layer * s.T + t0;
  uint32_t* sort_code = nullptr;         // per token: distance | position among the warp's tokens of that distance << 8
  {
    uint32_t* arena = dyn_smem + 2 * a.mask_words;
    if (a.stage_sorted) { sorted = reinterpret_cast<int32_t*>(arena); arena += a.stage_words; }
    if (a.stage_sig) {
      _Pragma("unroll 8") for (int i = tid; i < L * W; i += kThreads) arena[i] = __ldg(sig + i);
      sig = arena;
      arena += a.stage_words * W;
    }
    if (a.stage_keys) {
      unsigned long long* ks = reinterpret_cast<unsigned long long*>(arena);
      sort_code = reinterpret_cast<uint32_t*>(arena);      // the keys are dead once the important set is marked
      if (a.keys) {
        _Pragma("unroll 8") for (int i = tid; i < L; i += kThreads) ks[i] = keys[i];
      } else {
        const double* imp = a.imp + (size_t)layer * s.T + t0;
        _Pragma("unroll 8") for (int i = tid; i < L; i += kThreads) ks[i] = importance_key(__ldg(imp + i), i, L, a.keep_initial, a.keep_recent);
      }
      keys = ks;
    }
  }
  const int n_words = (L + 31) >> 5;
  int r_lo, r_hi;                            // contiguous token range of this warp
  sel::warp_range(L, warp, r_lo, r_hi);

  for (int i = tid; i < n_words; i += kThreads) { imp_mask[i] = 0; rep_mask[i] = 0; }
  __syncthreads();

  // ---- 1. important tokens: the b_imp largest keys, ties to the lower index --------------------
  if (b_imp > 0) sel::mark_top_keys(keys, L, b_imp, imp_mask, sc);

  // ---- 2-4. representatives of the other tokens ------------------------------------------------
  if (b_rep > 0) {
    const int N = L - b_imp;
    // anchor
    if (a.anchor_mode == KVCRUSH_ANCHOR_MEAN) {
      for (int i = tid; i < 128; i += kThreads) bit_cnt[i] = 0;
      __syncthreads();
      int acc[4] = {0, 0, 0, 0};
      for (int base = r_lo; base < r_hi; base += 32) {
        const int i = base + lane;
        const bool cand = i < r_hi && !((imp_mask[base >> 5] >> lane) & 1u);
        _Pragma("unroll") for (int w = 0; w < W; ++w) {
          const uint32_t word = cand ? sig[(size_t)i * W + w] : 0u;
          const int nb = min(32, s.Hq - 32 * w);
          for (int b = 0; b < nb; ++b) {
            const unsigned m = __ballot_sync(kFull, (word >> b) & 1u);
            if (lane == b) acc[w] += __popc(m);
          }
        }
      }
      _Pragma("unroll") for (int w = 0; w < W; ++w)
        if (32 * w + lane < s.Hq && acc[w]) atomicAdd(&bit_cnt[32 * w + lane], acc[w]);
      __syncthreads();
      if (warp < W) {
        const int h = 32 * warp + lane;
        const unsigned word = __ballot_sync(kFull, h < s.Hq && 2LL * bit_cnt[h] >= N);
        if (lane == 0) anchor_sh[warp] = word;
      }
    } else if (tid < W) {
      uint32_t word;
      if (a.anchor_mode == KVCRUSH_ANCHOR_EXPLICIT)
        word = __ldg(a.anchor_bits + (a.anchor_per_segment ? (size_t)seg * W : 0) + tid);
      else
        word = 0xAAAAAAAAu;
      anchor_sh[tid] = word & head_mask(s.Hq, tid);
    }
    for (int i = tid; i < kWarps * kMaxBins; i += kThreads) (&warp_hist[0][0])[i] = 0;
    __syncthreads();
    uint32_t anc[4], hm[4];
    _Pragma("unroll") for (int w = 0; w < 4; ++w) { anc[w] = w < W ? anchor_sh[w] : 0u; hm[w] = w < W ? head_mask(s.Hq, w) : 0u; }
    const int n_bins = s.Hq + 1;

    // counting sort by (d, t): per-warp histograms over contiguous token ranges.  When there is room, the first
    // sweep also notes every token's distance and its position among the warp's tokens of that distance, so that
    // the second sweep is a plain scatter.
    for (int base = r_lo; base < r_hi; base += 32) {
      const int i = base + lane;
      const bool cand = i < r_hi && !((imp_mask[base >> 5] >> lane) & 1u);
      int d = 0;
      if (cand)
        _Pragma("unroll") for (int w = 0; w < W; ++w) d += __popc((sig[(size_t)i * W + w] ^ anc[w]) & hm[w]);
      const unsigned voters = __ballot_sync(kFull, cand);
      unsigned peers = 0;
      if (cand) {
        peers = __match_any_sync(voters, d);
        if (sort_code) sort_code[i] = (uint32_t)d | ((uint32_t)(warp_hist[warp][d] + __popc(peers & lt_mask)) << 8);
      } else if (sort_code && i < r_hi) {
        sort_code[i] = 0xFFFFFFFFu;
      }
      __syncwarp();
      if (cand && (peers & lt_mask) == 0) warp_hist[warp][d] += __popc(peers);
      __syncwarp();
    }
    __syncthreads();
    if (tid < n_bins) {                     // per bin: exclusive prefix over warps (token order)
      int run = 0;
      for (int w = 0; w < kWarps; ++w) { const int c = warp_hist[w][tid]; warp_hist[w][tid] = run; run += c; }
      bin_base[tid + 1] = run;
    }
    __syncthreads();
    if (tid == 0) {
      bin_base[0] = 0;
      for (int b = 1; b <= n_bins; ++b) bin_base[b] += bin_base[b - 1];
    }
    __syncthreads();
    if (sort_code) {
      for (int i = r_lo + lane; i < r_hi; i += 32) {
        const uint32_t c = sort_code[i];
        if (c != 0xFFFFFFFFu) {
          const int d = (int)(c & 0xFFu);
          sorted[bin_base[d] + warp_hist[warp][d] + (int)(c >> 8)] = i;
        }
      }
    } else {
      for (int base = r_lo; base < r_hi; base += 32) {
        const int i = base + lane;
        const bool cand = i < r_hi && !((imp_mask[base >> 5] >> lane) & 1u);
        int d = 0;
        if (cand)
          _Pragma("unroll") for (int w = 0; w < W; ++w) d += __popc((sig[(size_t)i * W + w] ^ anc[w]) & hm[w]);
        const unsigned voters = __ballot_sync(kFull, cand);
        unsigned peers = 0;
        if (cand) {
          peers = __match_any_sync(voters, d);
          sorted[bin_base[d] + warp_hist[warp][d] + __popc(peers & lt_mask)] = i;
        }
        __syncwarp();
        if (cand && (peers & lt_mask) == 0) warp_hist[warp][d] += __popc(peers);
        __syncwarp();
      }
    }
    __syncthreads();

    // one representative per equal-frequency bucket
    // bucket i covers sorted positions [floor(i*N/R), floor((i+1)*N/R)); N = q_nr*R + r_nr
    const int q_nr = N / b_rep, r_nr = N - q_nr * b_rep;
    const int m_max = q_nr + (r_nr > 0 ? 1 : 0);                               // largest bucket
    if (m_max <= 16) {
      // Small buckets (the usual case: N/R is the compression ratio): 32 / gw buckets share a warp, gw = the power
      // of two that holds a bucket, one lane per member.  sum_{h set in t} n_h = sum over members u of
      // popc(sig_t & sig_u), so cost(t) = m * popc(sig_t) - 2 * sum_u popc(sig_t & sig_u): gw shuffles inside
      // the lane group.  |cost| <= 16 * 128 and t < 2^18, so (cost, t) packs into 31 bits and one warp-level
      // minimum per lane group picks the representative, ties to the lower token.
      int gw = 2;
      while (gw < m_max) gw <<= 1;
      const int per_warp = 32 / gw, sub = lane / gw, j = lane - sub * gw;
      const unsigned gmask = (0xFFFFFFFFu >> (32 - gw)) << (sub * gw);
      // bucket b starts at b*q_nr + frac with b*r_nr = frac*R + rem.  Divisions are slow, so each lane divides once
      // for its first bucket and then steps exactly by the warp's stride of kWarps*per_warp buckets.
      const int first_bkt = warp * per_warp + sub, stride_b = kWarps * per_warp;
      const unsigned long long p0 = (unsigned long long)(unsigned)first_bkt * (unsigned)r_nr;
      const unsigned long long ps = (unsigned long long)(unsigned)stride_b * (unsigned)r_nr;
      int frac = (int)(p0 / (unsigned)b_rep), rem = (int)(p0 - (unsigned long long)frac * (unsigned)b_rep);
      const int step_q = (int)(ps / (unsigned)b_rep), step_r = (int)(ps - (unsigned long long)step_q * (unsigned)b_rep);
      for (int bkt = first_bkt; bkt - sub < b_rep; bkt += stride_b) {
        const bool live = bkt < b_rep;
        const int lo = live ? bkt * q_nr + frac : 0;
        const int m = live ? q_nr + (rem + r_nr >= b_rep ? 1 : 0) : 0;       // the next bucket's frac is one larger
        frac += step_q;
        rem += step_r;
        if (rem >= b_rep) { rem -= b_rep; ++frac; }
        const bool member = j < m;
        const int t = member ? sorted[lo + j] : 0;
        uint32_t mine[4] = {0u, 0u, 0u, 0u};
        _Pragma("unroll") for (int w = 0; w < W; ++w) mine[w] = member ? sig[(size_t)t * W + w] & head_mask(s.Hq, w) : 0u;
        int ones = 0;
        _Pragma("unroll") for (int w = 0; w < W; ++w) ones += __popc(mine[w]);
        // lanes past a bucket's last member hold zeros and add nothing
        const int shared = gw == 8 ? group_and_popc<W, 8>(mine) : gw == 4 ? group_and_popc<W, 4>(mine)
                         : gw == 16 ? group_and_popc<W, 16>(mine) : group_and_popc<W, 2>(mine);
        const int cost = m * ones - 2 * shared;
        const uint32_t key = member ? ((uint32_t)(cost + 4096) << 18) | (uint32_t)t : 0xFFFFFFFFu;
        const uint32_t best = __reduce_min_sync(gmask, key);
        if (j == 0 && live) {
          const uint32_t bt = best & 0x3FFFFu;
          atomicOr(&rep_mask[bt >> 5], 1u << (bt & 31));
        }
      }
    } else {
    // Larger buckets: one warp per bucket.  64-bit divisions are slow, so each
    // warp divides once and then steps exactly: i*N = pos*R + rem, and the stride kWarps*N = step_q*R + step_r.
    const long long stride = (long long)kWarps * N;
    const int step_q = (int)(stride / b_rep), step_r = (int)(stride - (long long)step_q * b_rep);
    int pos = (int)(((long long)warp * N) / b_rep);
    int rem = (int)((long long)warp * N - (long long)pos * b_rep);
    for (int bkt = warp; bkt < b_rep; bkt += kWarps) {
      const int lo = pos;
      const int hi = pos + q_nr + (rem + r_nr >= b_rep ? 1 : 0);
      const int m = hi - lo;
      pos += step_q;
      rem += step_r;
      if (rem >= b_rep) { rem -= b_rep; ++pos; }
      unsigned long long best = ~0ull;
      if (m <= 32) {
        // one lane per member.  sum_{h set in t} n_h = sum over members u of popc(sig_t & sig_u), so
        // cost(t) = m * popc(sig_t) - 2 * sum_u popc(sig_t & sig_u): m shuffles instead of one ballot per head
        const bool member = lane < m;
        const int t = member ? sorted[lo + lane] : 0;
        uint32_t mine[4] = {0u, 0u, 0u, 0u};
        _Pragma("unroll") for (int w = 0; w < W; ++w) mine[w] = member ? sig[(size_t)t * W + w] & head_mask(s.Hq, w) : 0u;
        int ones = 0, shared = 0;
        _Pragma("unroll") for (int w = 0; w < W; ++w) ones += __popc(mine[w]);
        for (int u0 = 0; u0 < m; u0 += 4) {        // lanes >= m hold zeros, so reading past m adds nothing
          _Pragma("unroll") for (int du = 0; du < 4; ++du)
            _Pragma("unroll") for (int w = 0; w < W; ++w) shared += __popc(mine[w] & __shfl_sync(kFull, mine[w], (u0 + du) & 31));
        }
        const int cost = m * ones - 2 * shared;
        if (member) best = ((unsigned long long)((uint32_t)cost + 0x80000000u) << 32) | (uint32_t)t;
      } else {
        int n_ones[4] = {0, 0, 0, 0};        // lane b of word w holds n_h for head 32w+b
        for (int c0 = lo; c0 < hi; c0 += 32) {
          const bool member = c0 + lane < hi;
          const int t = member ? sorted[c0 + lane] : 0;
          _Pragma("unroll") for (int w = 0; w < W; ++w) {
            const uint32_t word = member ? sig[(size_t)t * W + w] : 0u;
            const int nb = min(32, s.Hq - 32 * w);
            for (int b = 0; b < nb; ++b) {
              const unsigned ones = __ballot_sync(kFull, (word >> b) & 1u);
              if (lane == b) n_ones[w] += __popc(ones);
            }
          }
        }
        for (int c0 = lo; c0 < hi; c0 += 32) {
          const bool member = c0 + lane < hi;
          const int t = member ? sorted[c0 + lane] : 0;
          int cost = 0;
          _Pragma("unroll") for (int w = 0; w < W; ++w) {
            const uint32_t word = member ? sig[(size_t)t * W + w] : 0u;
            const int nb = min(32, s.Hq - 32 * w);
            for (int b = 0; b < nb; ++b) {
              const int n_h = __shfl_sync(kFull, n_ones[w], b);
              if ((word >> b) & 1u) cost += m - 2 * n_h;
            }
          }
          if (member) {
            const unsigned long long key = ((unsigned long long)((uint32_t)cost + 0x80000000u) << 32) | (uint32_t)t;
            best = key < best ? key : best;
          }
        }
      }
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) {
        const unsigned long long o = __shfl_xor_sync(kFull, best, d);
        best = o < best ? o : best;
      }
      if (lane == 0) {
        const uint32_t t = (uint32_t)best;
        atomicOr(&rep_mask[t >> 5], 1u << (t & 31));
      }
    }
    }
    __syncthreads();
  }

  // ---- 5. kept = important U representatives, ascending ------------------------------------------
  sel::emit_kept(imp_mask, rep_mask, n_words, out_idx, out_kind, sc);
}

}  // namespace

int launch_importance(const Shape& s, const float* scores, int keep_initial, int keep_recent,
                      unsigned long long* keys, cudaStream_t stream) {
  const size_t n = (size_t)s.n_layers * s.T;
  importance_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(s, scores, keep_initial, keep_recent, keys);
  return check_launch();
}

int launch_importance_keys(const Shape& s, const double* importance, int keep_initial, int keep_recent,
                           unsigned long long* keys, cudaStream_t stream) {
  const size_t n = (size_t)s.n_layers * s.T;
  importance_keys_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(s, importance, keep_initial, keep_recent, keys);
  return check_launch();
}

size_t select_workspace_bytes(const Shape& s) {
  const size_t n = (size_t)s.n_layers * s.T;
  return ((n * 8 + 255) / 256) * 256 + ((n * 4 + 255) / 256) * 256;
}

int launch_select(const Shape& s, const float* scores, const double* importance, const uint32_t* sigs,
                  const int32_t* budget_imp,
                  const int32_t* budget_rep, int anchor_mode, const uint32_t* anchor_bits, int anchor_per_segment,
                  int keep_initial, int keep_recent, const int32_t* cu_kept, int32_t* idx, uint8_t* kind,
                  int32_t* n_kept, void* ws, cudaStream_t stream) {
  if (s.T == 0) {                                   // nothing but empty sequences: every segment keeps nothing
    if (n_kept && cudaMemsetAsync(n_kept, 0, (size_t)s.n_layers * s.n_seqs * sizeof(int32_t), stream) != cudaSuccess)
      return KVCRUSH_ERR_CUDA;
    return KVCRUSH_OK;
  }
  const size_t n = (size_t)s.n_layers * s.T;
  unsigned long long* keys = static_cast<unsigned long long*>(ws);
  int32_t* sorted = reinterpret_cast<int32_t*>(static_cast<unsigned char*>(ws) + ((n * 8 + 255) / 256) * 256);

  SelectArgs a{};
  a.sigs = sigs; a.budget_imp = budget_imp; a.budget_rep = budget_rep;
  a.anchor_mode = anchor_mode; a.anchor_bits = anchor_bits; a.anchor_per_segment = anchor_per_segment;
  a.cu_kept = cu_kept; a.idx = idx; a.kind = kind; a.n_kept = n_kept; a.sorted = sorted;
  a.mask_words = ((s.max_seqlen + 31) / 32 + 3) & ~3;
  a.stage_words = (s.max_seqlen + 3) & ~3;
  size_t dyn = (size_t)a.mask_words * 2 * sizeof(uint32_t);
  const size_t budget = 196 * 1024;     // dynamic shared memory this kernel may take (static part: ~27 KB)
  const size_t per_tok = (size_t)a.stage_words * sizeof(uint32_t);
  if (dyn + per_tok <= budget) { a.stage_sorted = 1; dyn += per_tok; }
  if (dyn + per_tok * s.W <= budget) { a.stage_sig = 1; dyn += per_tok * s.W; }
  if (dyn + 2 * per_tok <= budget) { a.stage_keys = 1; dyn += 2 * per_tok; }
  // importance keys: computed here from the scores, or taken from the caller's I(t) - converted while the segment
  // kernel stages them, or by a small kernel when the segments are too long to be staged
  if (!importance) {
    if (launch_importance(s, scores, keep_initial, keep_recent, keys, stream) != KVCRUSH_OK) return KVCRUSH_ERR_CUDA;
    a.keys = keys;
  }
  if (importance) {
    if (a.stage_keys) {
      a.imp = importance; a.keep_initial = keep_initial; a.keep_recent = keep_recent;
    } else {
      importance_keys_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(s, importance, keep_initial, keep_recent, keys);
      if (check_launch() != KVCRUSH_OK) return KVCRUSH_ERR_CUDA;
      a.keys = keys;
    }
  }
  if (dyn > 16 * 1024) {     // static + dynamic shared memory above the 48 KB default needs the opt-in
    cudaError_t e = cudaSuccess;
    switch (s.W) {
      case 1: e = cudaFuncSetAttribute(select_segment_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn); break;
      case 2: e = cudaFuncSetAttribute(select_segment_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn); break;
      case 3: e = cudaFuncSetAttribute(select_segment_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn); break;
      default: e = cudaFuncSetAttribute(select_segment_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn); break;
    }
    if (e != cudaSuccess) return KVCRUSH_ERR_CUDA;
  }
  const unsigned n_seg = (unsigned)(s.n_layers * s.n_seqs);
  switch (s.W) {
    case 1: select_segment_kernel<1><<<n_seg, kThreads, dyn, stream>>>(s, a); break;
    case 2: select_segment_kernel<2><<<n_seg, kThreads, dyn, stream>>>(s, a); break;
    case 3: select_segment_kernel<3><<<n_seg, kThreads, dyn, stream>>>(s, a); break;
    default: select_segment_kernel<4><<<n_seg, kThreads, dyn, stream>>>(s, a); break;
  }
  return check_launch();
}

}  // namespace kvc
