// Stage 1 on the 5th-generation tensor cores (tcgen05 + TMEM + TMA), bf16 Q/K, head_dim 64 or 128.
//
// Attention column sums (Algorithm 1 of the paper: A_h = softmax(Q_h K_h^T / sqrt(d_k)), then the
// per-token sum of A_h over the queries) without ever storing the S x S matrix: two sweeps that
// both recompute 128 x 128 logit tiles.
//
//   sweep 1 (kColsum = false)  one CTA per (layer, head, sequence, 128-query tile): S = Q_tile K^T,
//                              TMEM lane = query row, so each epilogue thread owns one row and keeps
//                              its running (max, sum) in registers  ->  lse2(j) = log2 sum_t 2^(s2(j,t))
//   sweep 2 (kColsum = true)   one CTA per (layer, head, sequence, 128-key tile): S^T = K_tile Q^T,
//                              TMEM lane = key, so each epilogue thread owns one key column and adds
//                              2^(s2 - lse2(j)) = A(j, t) over all query tiles in a register.
//                              No shuffles or atomics: one deterministic store per key.
//   s2 = q.k * softmax_scale * log2(e).
//
// CTA = 10 warps: warp 0 issues TMA loads (one lane), warp 1 allocates TMEM and issues tcgen05.mma
// (one lane), warps 2..9 are two epilogue groups of 128 threads that take alternate tiles, each
// reading its own 128-column TMEM accumulator, so the MMA of tile i+1 overlaps the exponentials of
// tile i.  The stationary operand stays in shared memory for the CTA's life; the streamed operand
// runs through a ring of 128B-swizzled stages.  Two CTAs fit one SM (96 KB shared memory, 256 TMEM
// columns each).  CTAs are ordered heaviest-first (causal rows/columns have 1..n tiles).
// Every barrier wait is bounded; on expiry the CTA flags status, drains its copies and exits.
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace kvc {

namespace {

constexpr int kTile = 128;               // rows of both operands per tile
#ifndef KVC_EPI_GROUPS
#define KVC_EPI_GROUPS 2
#endif
constexpr int kGroups = KVC_EPI_GROUPS;  // epilogue groups of 128 threads; tile i goes to group i % kGroups
constexpr int kEpiThreads = 128;         // per epilogue group
constexpr int kThreads = 64 + kGroups * kEpiThreads;
constexpr int kBufs = kGroups < 2 ? 2 : kGroups;         // 128-column fp32 accumulators in TMEM; tile i uses buffer i % kBufs
constexpr uint32_t kTmemCols = kBufs * 128;
constexpr int kCtasPerSm = kGroups > 2 ? 1 : 2;
#ifndef KVC_STAGES
#define KVC_STAGES (kGroups > 2 ? 5 : 2)
#endif
constexpr int kStages = KVC_STAGES;      // ring depth of the streamed operand

using namespace tc;

struct ScoreArgs {
  Shape s;
  float scale_log2;
  const float* lse;       // sweep 2: row log-sum-exp; value * lse_mul is in the log2 domain
  float lse_mul;
  float* lse2_out;        // sweep 1: log2-domain output [n_layers][Hq][T]
  float* lse_nat_out;     // sweep 1: optional natural-log copy
  float* scores;          // sweep 2 output
  int normalize;
  int max_tiles;          // ceil(max_seqlen / 128)
  int n_items;            // number of (sequence, tile) pairs
  int32_t* status;
};

template <int D>
struct SmemLayout {
  static constexpr int kTileBytes = kTile * D * 2;
  static constexpr int kBlockBytes = kTile * 128;            // one 64-element k-block of a tile
  static constexpr int kFixedOff = 0;
  static constexpr int kRingOff = kTileBytes;
  static constexpr int kAuxOff = kRingOff + kStages * kTileBytes;
  static constexpr int kAuxBytes = 12288;
  static constexpr int kTotal = kAuxOff + kAuxBytes + 1024;  // + slack to align the base to 1024
};

struct Aux {                         // lives at kAuxOff
  unsigned long long full[kStages];
  unsigned long long empty[kStages];
  unsigned long long fixed_full;
  unsigned long long acc_full[kBufs];
  unsigned long long acc_empty[kBufs];
  unsigned long long drain;
  uint32_t tmem_base;
  int abort_flag;
  int item[4];                       // seq, tile, n_tiles
  alignas(16) float lse_sh[kGroups][2][kTile];   // [group][buffer][query in tile]   (sweep 2)
  alignas(16) float part[kGroups][2][kTile];     // partials of groups 1.. handed to group 0
};

template <int D, bool kColsum>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
score_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const ScoreArgs a) {
  using SL = SmemLayout<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  Aux* aux = reinterpret_cast<Aux*>(smem + SL::kAuxOff);
  volatile int* abort_flag = &aux->abort_flag;
  const uint32_t fixed_addr = smem_u32(smem + SL::kFixedOff);
  const uint32_t ring_addr = smem_u32(smem + SL::kRingOff);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const Shape& s = a.s;
#ifdef KVC_RANK_MAJOR
  const int n_lh = s.n_layers * s.Hq;
#endif
  // Block order: all tile-rows of one (layer, head) are adjacent, heaviest first, so the CTAs that run
  // at the same time stream the same few heads' Q/K and those stay in L2.
#ifdef KVC_RANK_MAJOR
  const int lh = blockIdx.x % n_lh;
  const int rank = blockIdx.x / n_lh;
#else
  const int lh = blockIdx.x / a.n_items;
  const int rank = blockIdx.x - lh * a.n_items;
#endif
  const int layer = lh / s.Hq, h = lh - layer * s.Hq;
  const int hk = h / s.G;

  if (warp == 0) {
    int seq, tile, nt;
    decode_item(s.cu_seqlens, s.n_seqs, a.max_tiles, rank, !kColsum, lane, seq, tile, nt);
    if (lane == 0) {
      aux->item[0] = seq; aux->item[1] = tile; aux->item[2] = nt;
      // a launch that already failed somewhere is not worth finishing: later CTAs leave at once
      aux->abort_flag = *reinterpret_cast<volatile int32_t*>(a.status) != 0;
      for (int i = 0; i < kStages; ++i) { mbar_init(smem_u32(&aux->full[i]), 1); mbar_init(smem_u32(&aux->empty[i]), 1); }
      mbar_init(smem_u32(&aux->fixed_full), 1);
      mbar_init(smem_u32(&aux->drain), 1);
      for (int i = 0; i < kBufs; ++i) { mbar_init(smem_u32(&aux->acc_full[i]), 1); mbar_init(smem_u32(&aux->acc_empty[i]), 4); }
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
  } else if (warp == 1) {
    tmem_alloc(smem_u32(&aux->tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  const int seq = aux->item[0], my_tile = aux->item[1], n_tiles = aux->item[2];
  const uint32_t tmem_base = aux->tmem_base;
  const int t0 = __ldg(s.cu_seqlens + seq);
  const int L = __ldg(s.cu_seqlens + seq + 1) - t0;
  // tiles of the streamed operand swept by this CTA
  const int first_stream = kColsum ? (s.causal ? my_tile : 0) : 0;
  const int n_iter = s.causal ? (kColsum ? n_tiles - my_tile : my_tile + 1) : n_tiles;
  // sweep 1: A = Q tile (stationary), B = K tiles.  sweep 2: A = K tile (stationary), B = Q tiles.
  const CUtensorMap* map_fixed = kColsum ? &map_k : &map_q;
  const CUtensorMap* map_stream = kColsum ? &map_q : &map_k;
  const int head_fixed = kColsum ? hk : h, head_stream = kColsum ? h : hk;

  const bool dead = aux->abort_flag != 0;
  if (dead) {
    // nothing to do
  } else if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      mbar_expect_tx(smem_u32(&aux->fixed_full), SL::kTileBytes);
#pragma unroll
      for (int kb = 0; kb < D / 64; ++kb)
        tma_load_4d(fixed_addr + kb * SL::kBlockBytes, map_fixed, smem_u32(&aux->fixed_full), kb * 64,
                    t0 + my_tile * kTile, head_fixed, layer);
      int issued = 0;
      for (int it = 0; it < n_iter; ++it) {
        const int st = it % kStages;
        if (!mbar_wait(smem_u32(&aux->empty[st]), ((it / kStages) & 1) ^ 1, abort_flag)) break;
        mbar_expect_tx(smem_u32(&aux->full[st]), SL::kTileBytes);
#pragma unroll
        for (int kb = 0; kb < D / 64; ++kb)
          tma_load_4d(ring_addr + st * SL::kTileBytes + kb * SL::kBlockBytes, map_stream, smem_u32(&aux->full[st]),
                      kb * 64, t0 + (first_stream + it) * kTile, head_stream, layer);
        issued = it + 1;
      }
      if (*abort_flag) {
        // give the copies in flight a bounded time to land before the CTA's shared memory is released
        for (int it = max(0, issued - kStages); it < issued; ++it)
          for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(smem_u32(&aux->full[it % kStages]), (it / kStages) & 1); ++i) {}
        for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(smem_u32(&aux->fixed_full), 0); ++i) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(kTile, kTile);
      bool ok = mbar_wait(smem_u32(&aux->fixed_full), 0, abort_flag);
      for (int it = 0; ok && it < n_iter; ++it) {
        const int st = it % kStages, b = it % kBufs;
        ok = mbar_wait(smem_u32(&aux->full[st]), (it / kStages) & 1, abort_flag) &&
             mbar_wait(smem_u32(&aux->acc_empty[b]), ((it / kBufs) & 1) ^ 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + b * kTile;
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t off = (k >> 2) * SL::kBlockBytes + (k & 3) * 32;
          umma_bf16(d_tmem, smem_desc_sw128(fixed_addr + off), smem_desc_sw128(ring_addr + st * SL::kTileBytes + off),
                    idesc, k > 0);
        }
        umma_commit(smem_u32(&aux->empty[st]));
        umma_commit(smem_u32(&aux->acc_full[b]));
      }
      if (!ok) {
        // wait (bounded) until every MMA already issued has retired before TMEM and shared memory go away
        umma_commit(smem_u32(&aux->drain));
        for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(smem_u32(&aux->drain), 0); ++i) {}
      }
    }
  } else {
    // ------------------------------ epilogue groups ------------------------------
    const int g = (warp - 2) >> 2;                 // epilogue group of this warp
    const int quarter = warp & 3;                  // TMEM lanes this warp may read
    const int r = quarter * 32 + lane;             // row of the accumulator tile = TMEM lane
    const int gtid = r;                            // index inside the group (0..127)
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const float scale = a.scale_log2;
    const f32x2 scale2 = splat2(scale);
    bool ok = true;

    if constexpr (kColsum) {
      const float* lse_row = a.lse + ((size_t)layer * s.Hq + h) * s.T + t0;
      const float ninf = __int_as_float(0xFF800000);
      auto load_lse = [&](int it) {                 // minus lse2 of this thread's query of streamed tile `it` (-inf past the end)
        const int j = (first_stream + it) * kTile + gtid;
        return (it < n_iter && j < L) ? -(__ldg(lse_row + j) * a.lse_mul) : ninf;
      };
      f32x2 acc[2] = {0ull, 0ull};
      float lse_next = load_lse(g);
      int n_mine = 0;
      for (int it = g; it < n_iter; it += kGroups, ++n_mine) {
        const int b = it % kBufs;                   // TMEM accumulator of this tile
        float* lse_buf = aux->lse_sh[g][n_mine & 1];
        lse_buf[gtid] = lse_next;
        lse_next = load_lse(it + kGroups);          // in flight while this tile is processed
        named_bar_sync(1 + g, kEpiThreads);
        // after a failed wait the loop keeps running (every thread must reach every named barrier) but
        // touches neither barriers nor TMEM; `ok` is made warp-uniform because tcgen05.ld is warp-wide
        if (ok) ok = mbar_wait(smem_u32(&aux->acc_full[b]), (it / kBufs) & 1, abort_flag);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) continue;
        tc_fence_after();
        auto release = [&]() {                      // accumulator drained: hand it back to the MMA warp
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&aux->acc_empty[b]));
        };
        const uint32_t t_acc = t_lane + b * kTile;
        if (s.causal && it == 0)
          sweep_tile(t_acc, [&](const uint32_t (&v)[16], int p) { colsum_piece<true>(v, lse_buf + p * 16, scale2, r, p * 16, acc); }, release);
        else
          sweep_tile(t_acc, [&](const uint32_t (&v)[16], int p) { colsum_piece<false>(v, lse_buf + p * 16, scale2, r, p * 16, acc); }, release);
      }
      float total = sum4(acc);
      if constexpr (kGroups > 1) {
        if (g > 0) aux->part[g][0][r] = total;
        named_bar_sync(1 + kGroups, kGroups * kEpiThreads);
        if (g == 0)
          for (int o = 1; o < kGroups; ++o) total += aux->part[o][0][r];
      }
      if (g == 0 && ok && !*abort_flag) {
        const int t = my_tile * kTile + r;
        if (t < L) {
          if (a.normalize) total = total / (float)L;
          a.scores[((size_t)layer * s.Hq + h) * s.T + t0 + t] = total;
        }
      }
    } else {
      float m = __int_as_float(0xFF800000);                   // running max (log2 domain) of this row
      f32x2 sum2[2] = {0ull, 0ull};                           // packed partial sums of 2^(x - m)
      for (int it = g; it < n_iter; it += kGroups) {
        const int b = it % kBufs;
        ok = mbar_wait(smem_u32(&aux->acc_full[b]), (it / kBufs) & 1, abort_flag);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
        tc_fence_after();
        auto release = [&]() {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&aux->acc_empty[b]));
        };
        const uint32_t t_acc = t_lane + b * kTile;
        // keys of this tile that count for this row: up to the diagonal (causal) and inside the sequence
        const int n_valid = s.causal ? (it == my_tile ? r + 1 : kTile) : min(kTile, L - it * kTile);
        if (__any_sync(0xFFFFFFFFu, n_valid < kTile))
          sweep_tile(t_acc, [&](const uint32_t (&v)[16], int p) { lse_piece<true>(v, scale, scale2, n_valid - p * 16, m, sum2); }, release);
        else
          sweep_tile(t_acc, [&](const uint32_t (&v)[16], int p) { lse_piece<false>(v, scale, scale2, 16, m, sum2); }, release);
      }
      float sum = sum4(sum2);
      if constexpr (kGroups > 1) {
        if (g > 0) { aux->part[g][0][r] = m; aux->part[g][1][r] = sum; }
        named_bar_sync(1 + kGroups, kGroups * kEpiThreads);
        if (g == 0) {                               // merge the other groups' (max, sum)
          for (int o = 1; o < kGroups; ++o) {
            const float m1 = aux->part[o][0][r], sum1 = aux->part[o][1][r];
            const float big = fmaxf(m, m1);
            sum = sum * ex2(m - big) + (sum1 > 0.f ? sum1 * ex2(m1 - big) : 0.f);
            m = big;
          }
        }
      }
      if (g == 0 && ok && !*abort_flag) {
        const int j = my_tile * kTile + r;
        if (j < L) {
          const float lse2 = m + log2f(sum);
          const size_t o = ((size_t)layer * s.Hq + h) * s.T + t0 + j;
          a.lse2_out[o] = lse2;
          if (a.lse_nat_out) a.lse_nat_out[o] = lse2 * 0.69314718055994530942f;
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
  if (tid == 0 && !dead && *abort_flag) report(a.status, KVCRUSH_DEV_TIMEOUT, kColsum ? KID_SCORE_COLSUM : KID_SCORE_LSE, blockIdx.x, 0);
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
template <int D, bool kColsum>
int launch_sweep(const CUtensorMap& mq, const CUtensorMap& mk, const ScoreArgs& a, cudaStream_t stream) {
  auto kern = score_tc_kernel<D, kColsum>;
  constexpr int smem = SmemLayout<D>::kTotal;
  static bool configured = false;      // per process; the attribute is idempotent, so a race only repeats the call
  if (!configured) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return KVCRUSH_ERR_CUDA;
    configured = true;
  }
  const long long blocks = (long long)a.n_items * a.s.n_layers * a.s.Hq;
  if (blocks > 0x7FFFFFFFLL) return KVCRUSH_ERR_UNSUPPORTED;
  kern<<<(unsigned)blocks, kThreads, smem, stream>>>(mq, mk, a);
  return check_launch();
}

}  // namespace

bool score_tensor_supported(const Shape& s, const TensorView& Q, const TensorView& K) {
  if (Q.dtype != KVCRUSH_BF16 || K.dtype != KVCRUSH_BF16) return false;
  if (s.D != 64 && s.D != 128) return false;
  if (s.T < 1) return false;
  return encode_fn() != nullptr;
}

int launch_score_tensor(const Shape& s, const int32_t* cu_host, const TensorView& Q, const TensorView& K,
                        float scale_log2, const float* lse_in, float lse_in_mul, float* lse2_ws, float* scores,
                        float* lse_out, int normalize, int32_t* status, cudaStream_t stream) {
  static_assert(sizeof(Aux) <= 12288, "aux block too large");
  if (!(scale_log2 > 0.f)) return KVCRUSH_ERR_UNSUPPORTED;
  CUtensorMap mq, mk;
  if (!make_map(&mq, Q, s.D, s.T, s.Hq, s.n_layers) || !make_map(&mk, K, s.D, s.T, s.Hkv, s.n_layers))
    return KVCRUSH_ERR_CUDA;
  ScoreArgs a{};
  a.s = s; a.scale_log2 = scale_log2; a.normalize = normalize; a.status = status; a.scores = scores;
  a.max_tiles = (s.max_seqlen + kTile - 1) / kTile;
  long long items = 0;
  for (int i = 0; i < s.n_seqs; ++i) items += (cu_host[i + 1] - cu_host[i] + kTile - 1) / kTile;
  if (items == 0) return KVCRUSH_OK;
  if (items > 0x7FFFFFFF) return KVCRUSH_ERR_UNSUPPORTED;
  a.n_items = (int)items;
  int rc;
  if (!lse_in) {
    a.lse2_out = lse2_ws; a.lse_nat_out = lse_out;
    rc = s.D == 128 ? launch_sweep<128, false>(mq, mk, a, stream) : launch_sweep<64, false>(mq, mk, a, stream);
    if (rc != KVCRUSH_OK) return rc;
    a.lse = lse2_ws; a.lse_mul = 1.f;
  } else {
    a.lse = lse_in; a.lse_mul = lse_in_mul;
  }
  return s.D == 128 ? launch_sweep<128, true>(mq, mk, a, stream) : launch_sweep<64, true>(mq, mk, a, stream);
}

}  // namespace kvc
