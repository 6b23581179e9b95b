// Page- and chunk-granular KVCrush (Sec. 4.3.4: chunks of 8 tokens; Sec. 4.3.5: pages of 32 tokens).
// A page is page_size consecutive tokens of one sequence; the last page of a sequence may be short and its
// missing tokens count as all-zero vectors of zero importance.
//
//   importance of a page  = sum of the token importances I(t), float64, tokens added in ascending order
//   vector of a page      = the signatures of its tokens one after the other (page_size * W words)
//   anchor of a page      = the token anchor repeated in every slot (alternating / explicit), or the per-bit
//                           majority of the grouped pages (mean)
// and then the token-level steps with pages in the place of tokens: top budget_imp pages, Hamming distance of
// the others to the anchor, (distance, page) order cut into budget_rep equal-frequency buckets, one
// representative per bucket (integer L1 cost to the per-bit mean), kept = important U representatives.
//
// One CTA per (layer, sequence).  A sequence has at most kMaxPagesPerSeq pages, so the page keys, the sort keys
// and the masks all live in shared memory; the (distance, page) order is one bitonic sort of 32-bit keys; a
// bucket is handled by one warp with per-bit counters in shared memory.
#include "select_common.cuh"

namespace kvc {

namespace {

using sel::kThreads;
using sel::kWarps;
using sel::kFull;
using sel::head_mask;

struct PageArgs {
  const unsigned long long* tok_keys;  // [n_layers][T] order-preserving keys of I(t); or, when NULL,
  const double* tok_imp;               // [n_layers][T] I(t) itself, handed over by the caller
  const uint32_t* sigs;                // [n_layers][T][W]
  const int32_t* budget_imp;
  const int32_t* budget_rep;
  int anchor_mode;
  const uint32_t* anchor_bits;
  int anchor_per_segment;
  const int32_t* cu_kept;
  int32_t* page_idx;
  uint8_t* kind;
  int32_t* n_kept;                     // optional [n_layers][n_seqs]: pages kept per segment
  int P;                               // tokens per page
  int PW;                              // words per page vector = P * W
  int np_cap;                          // capacity of the per-page arrays (pages, multiple of 32)
  int sort_cap;                        // capacity of the sort array (power of two >= np_cap)
  int n_workers;                       // warps that own per-bit counters
  int keep_initial, keep_recent;       // pages at both ends of a sequence that are important by decree
};

__device__ __forceinline__ double key_to_double(unsigned long long k) {
  const unsigned long long b = (k >> 63) ? (k & 0x7FFFFFFFFFFFFFFFull) : ~k;
  return __longlong_as_double((long long)b);
}

__device__ __forceinline__ unsigned long long double_to_key(double v) {
  const unsigned long long b = (unsigned long long)__double_as_longlong(v);
  return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
}

__global__ void __launch_bounds__(kThreads, 1)
select_pages_kernel(Shape s, PageArgs a) {
  extern __shared__ __align__(16) unsigned char dyn_raw[];
  unsigned long long* pkeys = reinterpret_cast<unsigned long long*>(dyn_raw);        // [np_cap]
  uint32_t* skey = reinterpret_cast<uint32_t*>(pkeys + a.np_cap);                    // [sort_cap]
  uint32_t* imp_mask = skey + a.sort_cap;                                            // [np_cap / 32]
  uint32_t* rep_mask = imp_mask + a.np_cap / 32;                                     // [np_cap / 32]
  uint32_t* anchor = rep_mask + a.np_cap / 32;                                       // [PW]
  uint32_t* counters = anchor + a.PW;                                                // [n_workers][PW * 16] (u16 pairs)

  __shared__ sel::Scratch sc;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int seg = blockIdx.x;
  const int layer = seg / s.n_seqs, seq = seg - layer * s.n_seqs;
  const int t0 = __ldg(s.cu_seqlens + seq);
  const int L = __ldg(s.cu_seqlens + seq + 1) - t0;
  const int P = a.P, PW = a.PW, W = s.W;
  const int n_pages = (L + P - 1) / P;
  const int b_imp = max(0, __ldg(a.budget_imp + seg));
  const int b_rep = max(0, __ldg(a.budget_rep + seg));
  int32_t* out_idx = a.page_idx + __ldg(a.cu_kept + seg);
  uint8_t* out_kind = a.kind ? a.kind + __ldg(a.cu_kept + seg) : nullptr;

  if (a.n_kept && tid == 0) a.n_kept[seg] = (int)min((long long)b_imp + b_rep, (long long)n_pages);
  if ((long long)b_imp + b_rep >= n_pages) {       // budget covers the sequence: keep every page
    for (int i = tid; i < n_pages; i += kThreads) {
      out_idx[i] = i;
      if (out_kind) out_kind[i] = 0;
    }
    return;
  }

  const unsigned long long* tkeys = a.tok_keys ? a.tok_keys + (size_t)layer * s.T + t0 : nullptr;
  const double* timp = a.tok_imp ? a.tok_imp + (size_t)layer * s.T + t0 : nullptr;
  const uint32_t* sig = a.sigs + ((size_t)layer * s.T + t0) * W;
  const int n_words = (n_pages + 31) >> 5;

  // page importance (sequential float64 adds, tokens ascending) as an order-preserving key
  for (int p = tid; p < n_pages; p += kThreads) {
    const int first = p * P, n_tok = min(P, L - first);
    double acc = 0.0;
    for (int i0 = 0; i0 < n_tok; i0 += 8) {        // the adds are sequential by definition, the loads are not
      double vv[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        vv[j] = i0 + j >= n_tok ? 0.0 : timp ? timp[first + i0 + j] : key_to_double(tkeys[first + i0 + j]);
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (i0 + j < n_tok) acc = __dadd_rn(acc, vv[j]);
    }
    if (p < a.keep_initial || p >= n_pages - a.keep_recent) acc = __longlong_as_double(0x7FF0000000000000LL);
    pkeys[p] = double_to_key(acc);
  }
  for (int i = tid; i < n_words; i += kThreads) { imp_mask[i] = 0; rep_mask[i] = 0; }
  __syncthreads();

  if (b_imp > 0) sel::mark_top_keys(pkeys, n_pages, b_imp, imp_mask, sc);

  if (b_rep > 0) {
    const int N = n_pages - b_imp;
    // ---- anchor of a page -------------------------------------------------------------------------
    if (a.anchor_mode == KVCRUSH_ANCHOR_MEAN) {
      uint32_t* bit_cnt = counters;                 // PW * 32 counters (n_workers >= 2 guarantees the room)
      for (int i = tid; i < PW * 32; i += kThreads) bit_cnt[i] = 0;
      __syncthreads();
      for (int p = tid; p < n_pages; p += kThreads) {
        if ((imp_mask[p >> 5] >> (p & 31)) & 1u) continue;
        const int n_w = min(P, L - p * P) * W;
        const uint32_t* pv = sig + (size_t)p * PW;
        for (int w = 0; w < n_w; ++w) {
          uint32_t word = pv[w] & head_mask(s.Hq, w % W);
          while (word) {
            const int b = __ffs(word) - 1;
            word &= word - 1;
            atomicAdd(&bit_cnt[w * 32 + b], 1u);
          }
        }
      }
      __syncthreads();
      for (int w = warp; w < PW; w += kWarps) {
        const unsigned word = __ballot_sync(kFull, 2LL * bit_cnt[w * 32 + lane] >= N);
        if (lane == 0) anchor[w] = word & head_mask(s.Hq, w % W);
      }
    } else {
      for (int w = tid; w < PW; w += kThreads) {
        uint32_t word = 0xAAAAAAAAu;
        if (a.anchor_mode == KVCRUSH_ANCHOR_EXPLICIT)
          word = __ldg(a.anchor_bits + (a.anchor_per_segment ? (size_t)seg * W : 0) + w % W);
        anchor[w] = word & head_mask(s.Hq, w % W);
      }
    }
    __syncthreads();

    // ---- (distance, page) order of the grouped pages: bitonic sort of d << 16 | page ----------------
    int n_sort = 32;
    while (n_sort < n_pages) n_sort <<= 1;
    for (int p = tid; p < n_sort; p += kThreads) {
      uint32_t key = 0xFFFFFFFFu;                   // important pages and padding sort to the end
      if (p < n_pages && !((imp_mask[p >> 5] >> (p & 31)) & 1u)) {
        const int n_w = min(P, L - p * P) * W;
        const uint32_t* pv = sig + (size_t)p * PW;
        int d = 0;
        for (int w = 0; w < PW; ++w) {
          const uint32_t word = w < n_w ? pv[w] & head_mask(s.Hq, w % W) : 0u;
          d += __popc(word ^ anchor[w]);
        }
        key = ((uint32_t)d << 16) | (uint32_t)p;
      }
      skey[p] = key;
    }
    __syncthreads();
    for (int k = 2; k <= n_sort; k <<= 1) {
      for (int j = k >> 1; j > 0; j >>= 1) {
        for (int i = tid; i < n_sort; i += kThreads) {
          const int o = i ^ j;
          if (o > i) {
            const uint32_t x = skey[i], y = skey[o];
            const bool up = (i & k) == 0;
            if ((x > y) == up) { skey[i] = y; skey[o] = x; }
          }
        }
        __syncthreads();
      }
    }

    // ---- one representative per equal-frequency bucket (one warp per bucket) -------------------------
    if (warp < a.n_workers) {
      unsigned short* cnt = reinterpret_cast<unsigned short*>(counters) + (size_t)warp * PW * 32;
      for (int bkt = warp; bkt < b_rep; bkt += a.n_workers) {
        const int lo = (int)(((long long)bkt * N) / b_rep);
        const int hi = (int)(((long long)(bkt + 1) * N) / b_rep);
        const int m = hi - lo;
        for (int i = lane; i < PW * 32; i += 32) cnt[i] = 0;
        __syncwarp();
        // n_bit = number of members with that bit set: lane b owns bit b of every word
        for (int u = lo; u < hi; ++u) {
          const int p = (int)(skey[u] & 0xFFFFu);
          const int n_w = min(P, L - p * P) * W;
          const uint32_t* pv = sig + (size_t)p * PW;
          for (int w0 = 0; w0 < n_w; w0 += 32) {
            const uint32_t mine = w0 + lane < n_w ? pv[w0 + lane] & head_mask(s.Hq, (w0 + lane) % W) : 0u;
            const int nj = min(32, n_w - w0);
            for (int j = 0; j < nj; ++j) {
              const uint32_t word = __shfl_sync(kFull, mine, j);
              cnt[(w0 + j) * 32 + lane] += (word >> lane) & 1u;
            }
          }
        }
        __syncwarp();
        // cost of a member = sum over its set bits of (m - 2 n_bit)
        unsigned long long best = ~0ull;
        for (int u = lo; u < hi; ++u) {
          const int p = (int)(skey[u] & 0xFFFFu);
          const int n_w = min(P, L - p * P) * W;
          const uint32_t* pv = sig + (size_t)p * PW;
          int cost = 0;
          for (int w0 = 0; w0 < n_w; w0 += 32) {
            const uint32_t mine = w0 + lane < n_w ? pv[w0 + lane] & head_mask(s.Hq, (w0 + lane) % W) : 0u;
            const int nj = min(32, n_w - w0);
            for (int j = 0; j < nj; ++j) {
              const uint32_t word = __shfl_sync(kFull, mine, j);
              if ((word >> lane) & 1u) cost += m - 2 * (int)cnt[(w0 + j) * 32 + lane];
            }
          }
#pragma unroll
          for (int d = 16; d > 0; d >>= 1) cost += __shfl_xor_sync(kFull, cost, d);
          const unsigned long long key = ((unsigned long long)((uint32_t)cost + 0x80000000u) << 32) | (uint32_t)p;
          best = key < best ? key : best;
        }
        if (lane == 0) {
          const uint32_t p = (uint32_t)best;
          atomicOr(&rep_mask[p >> 5], 1u << (p & 31));
        }
        __syncwarp();
      }
    }
    __syncthreads();
  }

  sel::emit_kept(imp_mask, rep_mask, n_words, out_idx, out_kind, sc);
}

}  // namespace

int launch_select_pages(const Shape& s, const float* scores, const double* importance, const uint32_t* sigs,
                        int page_size,
                        const int32_t* budget_imp, const int32_t* budget_rep, int anchor_mode,
                        const uint32_t* anchor_bits, int anchor_per_segment, int keep_initial, int keep_recent,
                        const int32_t* cu_kept, int32_t* page_idx, uint8_t* kind, int32_t* n_kept, void* ws,
                        cudaStream_t stream) {
  if (s.T == 0) {                                   // nothing but empty sequences: every segment keeps nothing
    if (n_kept && cudaMemsetAsync(n_kept, 0, (size_t)s.n_layers * s.n_seqs * sizeof(int32_t), stream) != cudaSuccess)
      return KVCRUSH_ERR_CUDA;
    return KVCRUSH_OK;
  }
  unsigned long long* keys = static_cast<unsigned long long*>(ws);
  if (!importance && launch_importance(s, scores, 0, 0, keys, stream) != KVCRUSH_OK) return KVCRUSH_ERR_CUDA;

  PageArgs a{};
  a.tok_keys = importance ? nullptr : keys; a.tok_imp = importance; a.sigs = sigs; a.budget_imp = budget_imp; a.budget_rep = budget_rep;
  a.anchor_mode = anchor_mode; a.anchor_bits = anchor_bits; a.anchor_per_segment = anchor_per_segment;
  a.cu_kept = cu_kept; a.page_idx = page_idx; a.kind = kind; a.n_kept = n_kept;
  a.P = page_size; a.PW = page_size * s.W;
  a.keep_initial = keep_initial; a.keep_recent = keep_recent;
  const int max_pages = (s.max_seqlen + page_size - 1) / page_size;
  a.np_cap = ((max_pages + 31) / 32) * 32;
  a.sort_cap = 32;
  while (a.sort_cap < a.np_cap) a.sort_cap <<= 1;
  const size_t fixed = (size_t)a.np_cap * 8 + (size_t)a.sort_cap * 4 + (size_t)a.np_cap / 32 * 8 + (size_t)a.PW * 4;
  const size_t per_worker = (size_t)a.PW * 32 * sizeof(unsigned short);
  const size_t budget = 212 * 1024;       // dynamic shared memory this kernel may take (static part: ~10 KB)
  a.n_workers = (int)((budget - fixed) / per_worker);
  if (a.n_workers > sel::kWarps) a.n_workers = sel::kWarps;
  if (a.n_workers < 2) return KVCRUSH_ERR_UNSUPPORTED;
  const size_t dyn = fixed + per_worker * a.n_workers;
  if (dyn > 48 * 1024 &&
      cudaFuncSetAttribute(select_pages_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
    return KVCRUSH_ERR_CUDA;
  select_pages_kernel<<<(unsigned)(s.n_layers * s.n_seqs), kThreads, dyn, stream>>>(s, a);
  return check_launch();
}

}  // namespace kvc
