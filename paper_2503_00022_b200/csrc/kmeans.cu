// Clustering baseline of the paper's ablation "KMeans vs KVCrush" (Fig. 3: k-means with 100 iterations takes the
// place of Algorithm 2's anchor / bucket grouping).  Not part of the compression pass: it exists so that the cost of
// a conventional clustering of the same binary head vectors can be timed beside kvcrush_select.
//
// Lloyd's algorithm on the vectors of the tokens that are not important, k = budget_rep clusters per segment:
//   centroid c = (n_{c,h} / m_c)_h, kept as integers (bit counts n and member count m);
//   distance^2(b, c) = (sum_h n_h^2 + m * sum_{h: b_h = 1} (m - 2 n_h)) / m^2, compared exactly by cross-multiplying
//   64-bit integers; ties go to the lower cluster; a cluster without members keeps its centroid.
// The dot product sum_{h in b} n_h is evaluated on bit planes of the counts: plane p of cluster c has bit h set when
// bit p of n_{c,h} is set, so the sum is sum_p 2^p popc(b & plane_p); a cluster of m members needs only
// ceil(log2(m + 1)) planes, and clusters are small on average (N / k members).
//
//   kmeans_prepare_kernel   one block per segment: important set (the same exact top-k as kvcrush_select), the other
//                           tokens listed in ascending order, initial centroids = the vectors at ranks floor(i*N/k)
//   kmeans_assign_kernel    one thread per grouped token, clusters staged through shared memory in tiles; mode 1 also
//                           accumulates the next centroids (global integer atomics: order does not matter), mode 2
//                           votes for each cluster's member closest to the centroid (integer cost, ties to the lower
//                           token: one 64-bit atomic minimum)
//   kmeans_update_kernel    one thread per cluster: takes over the accumulated counts, rebuilds planes and sum n^2
//   kmeans_finish_kernel    one block per segment: representatives, the unused budget of empty clusters filled with
//                           the most important remaining tokens, kept list in ascending order
#include "select_common.cuh"

namespace kvc {

namespace {

using sel::kThreads;
using sel::kFull;

constexpr int kPlanes = 16;            // bit planes of a count: counts up to 65535 (segments of up to 32768 tokens)
constexpr int kTile = 64;              // clusters staged in shared memory at a time
constexpr int kAssignThreads = 256;

struct KmLayout {                       // offsets into the workspace, in bytes
  size_t keys, cand, assign, seg, cnt[2], m[2], planes, S, np, winner, total;
};

KmLayout km_layout(const Shape& s, int K) {
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  const size_t n = (size_t)s.n_layers * s.T, n_seg = (size_t)s.n_layers * s.n_seqs, HW = 32 * (size_t)s.W;
  KmLayout l{};
  size_t o = 0;
  l.keys = o; o += up(n * 8);
  l.cand = o; o += up(n * 4);
  l.assign = o; o += up(n * 4);
  l.seg = o; o += up(n_seg * 4 * sizeof(int));
  for (int i = 0; i < 2; ++i) { l.cnt[i] = o; o += up(n_seg * K * HW * 4); }
  for (int i = 0; i < 2; ++i) { l.m[i] = o; o += up(n_seg * K * 4); }
  l.planes = o; o += up(n_seg * K * kPlanes * s.W * 4);
  l.S = o; o += up(n_seg * K * 8);
  l.np = o; o += up(n_seg * K * 4);
  l.winner = o; o += up(n_seg * K * 8);
  l.total = o;
  return l;
}

struct KmArgs {
  unsigned long long* keys;      // [n_layers][T] importance keys (reps are zeroed by the finish kernel)
  int32_t* cand;                 // [n_layers][T] grouped tokens of each segment, ascending, at the segment's offset
  int32_t* assign;               // cluster of the grouped token at the same position
  int32_t* seg;                  // [n_seg][4]: N (0: nothing to cluster), k, b_imp, keep-all flag
  int32_t* cnt_cur; int32_t* cnt_acc;   // [n_seg][K][32 W] bit counts
  int32_t* m_cur; int32_t* m_acc;       // [n_seg][K]
  uint32_t* planes;              // [n_seg][K][kPlanes][W]
  long long* S;                  // [n_seg][K] sum_h n_h^2
  int32_t* np;                   // [n_seg][K] planes in use
  unsigned long long* winner;    // [n_seg][K] (cost, token) of the best member; all ones: no member
  const uint32_t* sigs;
  const int32_t* budget_imp; const int32_t* budget_rep;
  const int32_t* cu_kept; int32_t* idx; uint8_t* kind; int32_t* n_kept;
  int K;
  int mask_words;
  int32_t* status;
};

// planes, plane count and sum of squares of one cluster from its counts
__device__ __forceinline__ void rebuild_cluster(const Shape& s, const int32_t* cnt, int m, uint32_t* planes,
                                                long long* S, int32_t* np) {
  long long sq = 0;
  const int used = 32 - __clz(m);                            // n_h <= m
  for (int w = 0; w < s.W; ++w) {
    uint32_t pl[kPlanes];
#pragma unroll
    for (int p = 0; p < kPlanes; ++p) pl[p] = 0;
    for (int b = 0; b < 32; ++b) {
      const int v = cnt[32 * w + b];
      sq += (long long)v * v;
#pragma unroll
      for (int p = 0; p < kPlanes; ++p) pl[p] |= (uint32_t)((v >> p) & 1) << b;
    }
#pragma unroll
    for (int p = 0; p < kPlanes; ++p) planes[p * s.W + w] = pl[p];
  }
  *S = sq;
  *np = used;
}

__global__ void __launch_bounds__(kThreads, 1)
kmeans_prepare_kernel(Shape s, KmArgs a) {
  extern __shared__ uint32_t dyn_smem[];
  uint32_t* imp_mask = dyn_smem;
  uint32_t* grp_mask = dyn_smem + a.mask_words;
  uint32_t* zero_mask = dyn_smem + 2 * a.mask_words;
  __shared__ sel::Scratch sc;
  const int tid = threadIdx.x;
  const int seg = blockIdx.x;
  const int layer = seg / s.n_seqs, seq = seg - layer * s.n_seqs;
  const int t0 = __ldg(s.cu_seqlens + seq);
  const int L = __ldg(s.cu_seqlens + seq + 1) - t0;
  const int b_imp = max(0, __ldg(a.budget_imp + seg));
  int b_rep = max(0, __ldg(a.budget_rep + seg));
  int32_t* info = a.seg + 4 * seg;
  if (b_rep > a.K) {                                         // the caller promised budgets of at most K
    if (tid == 0) {
      report(a.status, KVCRUSH_DEV_BUDGET, KID_KMEANS, seg, b_rep);
      info[0] = 0; info[1] = 0; info[2] = 0; info[3] = 1;
    }
    return;
  }
  if (a.n_kept && tid == 0) a.n_kept[seg] = (int)min((long long)b_imp + b_rep, (long long)L);
  if ((long long)b_imp + b_rep >= L) {                       // the budget covers the sequence: keep everything
    int32_t* out_idx = a.idx + __ldg(a.cu_kept + seg);
    uint8_t* out_kind = a.kind ? a.kind + __ldg(a.cu_kept + seg) : nullptr;
    for (int i = tid; i < L; i += kThreads) {
      out_idx[i] = i;
      if (out_kind) out_kind[i] = 0;
    }
    if (tid == 0) { info[0] = 0; info[1] = 0; info[2] = b_imp; info[3] = 1; }
    return;
  }
  const unsigned long long* keys = a.keys + (size_t)layer * s.T + t0;
  const int n_words = (L + 31) >> 5;
  for (int i = tid; i < n_words; i += kThreads) { imp_mask[i] = 0; zero_mask[i] = 0; }
  __syncthreads();
  if (b_imp > 0) sel::mark_top_keys(keys, L, b_imp, imp_mask, sc);
  const int N = L - b_imp;
  for (int i = tid; i < n_words; i += kThreads) {
    const uint32_t valid = (i == n_words - 1 && (L & 31)) ? ((1u << (L & 31)) - 1u) : 0xFFFFFFFFu;
    grp_mask[i] = ~imp_mask[i] & valid;
  }
  __syncthreads();
  int32_t* cand = a.cand + (size_t)layer * s.T + t0;
  sel::emit_kept(grp_mask, zero_mask, n_words, cand, nullptr, sc);   // grouped tokens in ascending order
  if (tid == 0) { info[0] = b_rep > 0 ? N : 0; info[1] = b_rep; info[2] = b_imp; info[3] = 0; }
  __syncthreads();
  // initial centroids: the vectors at ranks floor(i * N / k)
  const uint32_t* sig = a.sigs + ((size_t)layer * s.T + t0) * s.W;
  const size_t cbase = (size_t)seg * a.K;
  for (int c = tid; c < b_rep; c += kThreads) {
    const int t = cand[(int)(((long long)c * N) / b_rep)];
    int32_t* cnt = a.cnt_cur + (cbase + c) * 32 * s.W;
    for (int w = 0; w < s.W; ++w) {
      const uint32_t word = sig[(size_t)t * s.W + w] & sel::head_mask(s.Hq, w);
      for (int b = 0; b < 32; ++b) cnt[32 * w + b] = (word >> b) & 1u;
    }
    a.m_cur[cbase + c] = 1;
    rebuild_cluster(s, cnt, 1, a.planes + (cbase + c) * kPlanes * s.W, a.S + cbase + c, a.np + cbase + c);
  }
}

// kMode 0: assign only; 1: assign and accumulate the next centroids; 2: assign and vote for each cluster's closest member
template <int W, int kMode>
__global__ void __launch_bounds__(kAssignThreads)
kmeans_assign_kernel(Shape s, KmArgs a) {
  __shared__ uint32_t pl_sh[kTile][kPlanes][W];
  __shared__ long long S_sh[kTile];
  __shared__ int m_sh[kTile], np_sh[kTile];
  const int seg = blockIdx.y;
  const int N = a.seg[4 * seg], k = a.seg[4 * seg + 1];
  const int r0 = blockIdx.x * kAssignThreads;
  if (r0 >= N) return;                                       // uniform over the block
  const int r = r0 + threadIdx.x;
  const bool live = r < N;
  const int layer = seg / s.n_seqs, seq = seg - layer * s.n_seqs;
  const int t0 = __ldg(s.cu_seqlens + seq);
  const size_t tbase = (size_t)layer * s.T + t0;
  const size_t cbase = (size_t)seg * a.K;
  const int t = live ? a.cand[tbase + r] : 0;
  uint32_t b[W];
  int pb = 0;
#pragma unroll
  for (int w = 0; w < W; ++w) {
    b[w] = live ? __ldg(a.sigs + (tbase + t) * W + w) & sel::head_mask(s.Hq, w) : 0u;
    pb += __popc(b[w]);
  }
  long long best_num = 0, best_den = 1, best_dot = 0;
  int best_c = -1, best_m = 1;
  for (int c0 = 0; c0 < k; c0 += kTile) {
    const int nc = min(kTile, k - c0);
    __syncthreads();
    for (int i = threadIdx.x; i < nc * kPlanes * W; i += kAssignThreads)
      (&pl_sh[0][0][0])[i] = a.planes[(cbase + c0) * kPlanes * W + i];
    for (int i = threadIdx.x; i < nc; i += kAssignThreads) {
      S_sh[i] = a.S[cbase + c0 + i];
      m_sh[i] = a.m_cur[cbase + c0 + i];
      np_sh[i] = a.np[cbase + c0 + i];
    }
    __syncthreads();
    for (int c = 0; c < nc; ++c) {
      const int np = np_sh[c];
      int dot = 0;
      for (int p = 0; p < np; ++p)
#pragma unroll
        for (int w = 0; w < W; ++w) dot += __popc(b[w] & pl_sh[c][p][w]) << p;
      const long long m = m_sh[c];
      const long long num = S_sh[c] + m * (m * pb - 2LL * dot);          // distance^2 = num / m^2
      const long long den = m * m;
      if (best_c < 0 || num * best_den < best_num * den) {
        best_num = num; best_den = den; best_c = c0 + c; best_dot = dot; best_m = (int)m;
      }
    }
  }
  if (!live) return;
  a.assign[tbase + r] = best_c;
  if (kMode == 1) {
    atomicAdd(a.m_acc + cbase + best_c, 1);
    int32_t* cnt = a.cnt_acc + (cbase + best_c) * 32 * W;
#pragma unroll
    for (int w = 0; w < W; ++w) {
      uint32_t word = b[w];
      while (word) {
        const int h = __ffs(word) - 1;
        word &= word - 1;
        atomicAdd(cnt + 32 * w + h, 1);
      }
    }
  }
  if (kMode == 2) {
    // closest member of the cluster: sum_{h in b} (m - 2 n_h) = m * popc(b) - 2 * dot, ties to the lower token
    const long long cost = (long long)best_m * pb - 2LL * best_dot;     // |cost| <= 128 * 32768 = 2^22
    const unsigned long long key = ((unsigned long long)(cost + (1LL << 23)) << 18) | (unsigned long long)(uint32_t)t;
    atomicMin(a.winner + cbase + best_c, key);
  }
}

__global__ void __launch_bounds__(256)
kmeans_update_kernel(Shape s, KmArgs a) {
  const int seg = blockIdx.y;
  const int c = blockIdx.x * 256 + threadIdx.x;
  if (c >= a.seg[4 * seg + 1] || a.seg[4 * seg] == 0) return;
  const size_t ci = (size_t)seg * a.K + c;
  const int m = a.m_acc[ci];
  if (m == 0) return;                                        // no member: the centroid stays
  int32_t* cur = a.cnt_cur + ci * 32 * s.W;
  const int32_t* acc = a.cnt_acc + ci * 32 * s.W;
  for (int i = 0; i < 32 * s.W; ++i) cur[i] = acc[i];
  a.m_cur[ci] = m;
  rebuild_cluster(s, cur, m, a.planes + ci * kPlanes * s.W, a.S + ci, a.np + ci);
}

__global__ void __launch_bounds__(kThreads, 1)
kmeans_finish_kernel(Shape s, KmArgs a) {
  extern __shared__ uint32_t dyn_smem[];
  uint32_t* imp_mask = dyn_smem;
  uint32_t* rep_mask = dyn_smem + a.mask_words;
  __shared__ sel::Scratch sc;
  __shared__ int n_reps;
  const int tid = threadIdx.x;
  const int seg = blockIdx.x;
  const int32_t* info = a.seg + 4 * seg;
  if (info[3]) return;                                       // everything was kept by the prepare kernel
  const int layer = seg / s.n_seqs, seq = seg - layer * s.n_seqs;
  const int t0 = __ldg(s.cu_seqlens + seq);
  const int L = __ldg(s.cu_seqlens + seq + 1) - t0;
  const int k = info[1], b_imp = info[2];
  unsigned long long* keys = a.keys + (size_t)layer * s.T + t0;
  const int n_words = (L + 31) >> 5;
  for (int i = tid; i < n_words; i += kThreads) { imp_mask[i] = 0; rep_mask[i] = 0; }
  if (tid == 0) n_reps = 0;
  __syncthreads();
  int mine = 0;
  for (int c = tid; c < k; c += kThreads) {
    const unsigned long long w = a.winner[(size_t)seg * a.K + c];
    if (w != ~0ull) {
      const uint32_t t = (uint32_t)(w & 0x3FFFFull);
      atomicOr(&rep_mask[t >> 5], 1u << (t & 31));
      keys[t] = 0ull;                                        // below every real key: never among the top ones
      ++mine;
    }
  }
  if (mine) atomicAdd(&n_reps, mine);
  __syncthreads();
  // the important set plus, for the budget that empty clusters left, the most important of the remaining tokens
  const int k_top = b_imp + (k - n_reps);
  if (k_top > 0) sel::mark_top_keys(keys, L, k_top, imp_mask, sc);
  __syncthreads();
  int32_t* out_idx = a.idx + __ldg(a.cu_kept + seg);
  uint8_t* out_kind = a.kind ? a.kind + __ldg(a.cu_kept + seg) : nullptr;
  sel::emit_kept(imp_mask, rep_mask, n_words, out_idx, out_kind, sc);
}

template <int kMode>
void launch_assign(const Shape& s, const KmArgs& a, dim3 grid, cudaStream_t stream) {
  switch (s.W) {
    case 1: kmeans_assign_kernel<1, kMode><<<grid, kAssignThreads, 0, stream>>>(s, a); break;
    case 2: kmeans_assign_kernel<2, kMode><<<grid, kAssignThreads, 0, stream>>>(s, a); break;
    case 3: kmeans_assign_kernel<3, kMode><<<grid, kAssignThreads, 0, stream>>>(s, a); break;
    default: kmeans_assign_kernel<4, kMode><<<grid, kAssignThreads, 0, stream>>>(s, a); break;
  }
}

}  // namespace

size_t kmeans_workspace_bytes(const Shape& s, int max_budget_rep) { return km_layout(s, max_budget_rep > 0 ? max_budget_rep : 1).total; }

bool kmeans_supported(const Shape& s) {
  // the exact comparison multiplies a numerator below 2 Hq m^2 by another cluster's m'^2 with m + m' <= L:
  // 2 Hq (L/2)^4 must stay below 2^63
  const long double l4 = (long double)s.max_seqlen * s.max_seqlen * (long double)s.max_seqlen * s.max_seqlen;
  return s.max_seqlen <= 32768 && (long double)s.Hq * l4 < 73786976294838206464.0L;     // 2^66
}

int launch_kmeans_select(const Shape& s, const float* scores, const double* importance, const uint32_t* sigs,
                         const int32_t* budget_imp, const int32_t* budget_rep, int max_budget_rep, int iterations,
                         int keep_initial, int keep_recent, const int32_t* cu_kept, int32_t* idx, uint8_t* kind,
                         int32_t* n_kept, void* ws, int32_t* status, cudaStream_t stream) {
  const int n_seg = s.n_layers * s.n_seqs;
  if (s.T == 0) {
    if (n_kept && cudaMemsetAsync(n_kept, 0, (size_t)n_seg * sizeof(int32_t), stream) != cudaSuccess) return KVCRUSH_ERR_CUDA;
    return KVCRUSH_OK;
  }
  const int K = max_budget_rep > 0 ? max_budget_rep : 1;
  const KmLayout l = km_layout(s, K);
  unsigned char* base = static_cast<unsigned char*>(ws);
  KmArgs a{};
  a.keys = reinterpret_cast<unsigned long long*>(base + l.keys);
  a.cand = reinterpret_cast<int32_t*>(base + l.cand);
  a.assign = reinterpret_cast<int32_t*>(base + l.assign);
  a.seg = reinterpret_cast<int32_t*>(base + l.seg);
  a.planes = reinterpret_cast<uint32_t*>(base + l.planes);
  a.S = reinterpret_cast<long long*>(base + l.S);
  a.np = reinterpret_cast<int32_t*>(base + l.np);
  a.winner = reinterpret_cast<unsigned long long*>(base + l.winner);
  a.sigs = sigs; a.budget_imp = budget_imp; a.budget_rep = budget_rep;
  a.cu_kept = cu_kept; a.idx = idx; a.kind = kind; a.n_kept = n_kept;
  a.K = K;
  a.status = status;
  a.mask_words = ((s.max_seqlen + 31) / 32 + 3) & ~3;
  int cur = 0;
  auto bind = [&]() {
    a.cnt_cur = reinterpret_cast<int32_t*>(base + l.cnt[cur]);
    a.cnt_acc = reinterpret_cast<int32_t*>(base + l.cnt[cur ^ 1]);
    a.m_cur = reinterpret_cast<int32_t*>(base + l.m[cur]);
    a.m_acc = reinterpret_cast<int32_t*>(base + l.m[cur ^ 1]);
  };
  bind();

  int rc = importance ? launch_importance_keys(s, importance, keep_initial, keep_recent, a.keys, stream)
                      : launch_importance(s, scores, keep_initial, keep_recent, a.keys, stream);
  if (rc != KVCRUSH_OK) return rc;
  const size_t dyn = (size_t)a.mask_words * 3 * sizeof(uint32_t);
  if (dyn > 16 * 1024) {
    if (cudaFuncSetAttribute(kmeans_prepare_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess ||
        cudaFuncSetAttribute(kmeans_finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
      return KVCRUSH_ERR_CUDA;
  }
  kmeans_prepare_kernel<<<n_seg, kThreads, dyn, stream>>>(s, a);
  if (check_launch() != KVCRUSH_OK) return KVCRUSH_ERR_CUDA;

  const dim3 grid_a((unsigned)((s.max_seqlen + kAssignThreads - 1) / kAssignThreads), (unsigned)n_seg);
  const dim3 grid_u((unsigned)((K + 255) / 256), (unsigned)n_seg);
  const size_t cnt_bytes = (size_t)n_seg * K * 32 * s.W * 4, m_bytes = (size_t)n_seg * K * 4;
  for (int it = 0; it < iterations; ++it) {
    // the accumulators are the other half of the double buffer; the update kernel copies what has members into
    // the current half, so the halves never swap
    if (cudaMemsetAsync(a.cnt_acc, 0, cnt_bytes, stream) != cudaSuccess ||
        cudaMemsetAsync(a.m_acc, 0, m_bytes, stream) != cudaSuccess)
      return KVCRUSH_ERR_CUDA;
    launch_assign<1>(s, a, grid_a, stream);
    if (check_launch() != KVCRUSH_OK) return KVCRUSH_ERR_CUDA;
    kmeans_update_kernel<<<grid_u, 256, 0, stream>>>(s, a);
    if (check_launch() != KVCRUSH_OK) return KVCRUSH_ERR_CUDA;
  }
  if (cudaMemsetAsync(a.winner, 0xFF, (size_t)n_seg * K * 8, stream) != cudaSuccess) return KVCRUSH_ERR_CUDA;
  launch_assign<2>(s, a, grid_a, stream);
  if (check_launch() != KVCRUSH_OK) return KVCRUSH_ERR_CUDA;
  kmeans_finish_kernel<<<n_seg, kThreads, dyn, stream>>>(s, a);
  return check_launch();
}

}  // namespace kvc
