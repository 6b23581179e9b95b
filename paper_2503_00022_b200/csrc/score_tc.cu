// Stage 1 on the 5th-generation tensor cores (tcgen05 + TMEM + TMA), bf16 or fp16 Q/K, head_dim up to 128
// (a multiple of 8; widths other than 64 and 128 run in the next larger kernel: the TMA boxes read zeros past
// the last channel, and zeros add nothing to a dot product).
//
// Attention column sums (Algorithm 1 of the paper: A_h = softmax(Q_h K_h^T / sqrt(d_k)), then the per-token
// sum of A_h over the queries) without ever storing the S x S matrix: two sweeps that both recompute
// 128 x 128 logit tiles.
//
//   sweep 1 (kColsum = false)  S = Q_block K^T: TMEM lane = query row, so each epilogue thread owns one row
//                              and keeps its running (max, sum) in registers -> lse2(j) = log2 sum_t 2^(s2(j,t))
//   sweep 2 (kColsum = true)   S^T = K_block Q^T: TMEM lane = key, so each epilogue thread owns one key column
//                              and adds 2^(s2 - lse2(j)) = A(j, t) over all query tiles in registers.
//                              No shuffles or atomics: one deterministic store per key.
//   s2 = q.k * softmax_scale * log2(e).
//
// On this part the sweeps run against the board's power limit, so the work decomposition is built to
// spend little energy per logit tile:
//
//   * one CTA per SM lives for the whole launch and pulls work items from an atomic counter, so TMEM
//     allocation, barrier set-up and pipeline fill are paid once per SM instead of once per item;
//   * an item is a 512-row block of the stationary operand (four 128-row quarters).  Every streamed
//     128-row tile is multiplied with all four quarters, which quarters the L2 -> shared-memory traffic per
//     logit compared with one tile pair per load;
//   * TMEM holds one 128-column accumulator per quarter, owned by one epilogue group: a group needs no merge
//     with another group, and while it waits for its accumulator to be refilled the other three keep the
//     special-function unit busy.
//
// Roles: warp 0 fetches + decodes items and issues TMA loads; warps 1 and 2 (one lane each) issue the
// tcgen05.mma of quarters 0-1 and 2-3; warps 3..18 are four epilogue groups (one per quarter) of 128 threads,
// thread = TMEM lane = one query row (sweep 1) or one key column (sweep 2).  All synchronisation is by mbarriers
// with bounded waits: a role that gives up sets the CTA's abort flag, every other wait then ends, the CTA
// reports through the status word, drains its copies, frees TMEM and returns.
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace kvc {

namespace {

using namespace tc;

constexpr int kTile = 128;
constexpr int kQ = 4;                        // stationary 128-row quarters per work item
constexpr int kBlockRows = kQ * kTile;       // stationary rows per work item
constexpr int kEpiWarps = 16;
#ifndef KVC_ISSUE_WARPS
#define KVC_ISSUE_WARPS 2
#endif
constexpr int kIssueWarps = KVC_ISSUE_WARPS;   // tcgen05.mma issuing threads; each owns kQ / kIssueWarps quarters
constexpr int kQPerIssuer = kQ / kIssueWarps;
constexpr int kThreads = 32 * (1 + kIssueWarps) + kEpiWarps * 32;
constexpr int kRing = 2;                     // streamed tiles in flight
constexpr uint32_t kTmemCols = 512;          // one 128-column fp32 accumulator per quarter
constexpr int kLseChunk = 16;                // sweep 2: streamed tiles whose row log-sum-exp is staged at once

struct PersistArgs {
  Shape s;
  float scale_log2;
  const float* lse;        // sweep 2: row log-sum-exp; value * lse_mul is in the log2 domain
  float lse_mul;
  float* lse2_out;         // sweep 1 output (log2 domain), [n_layers][Hq][T]
  float* lse_nat_out;      // sweep 1: optional natural-log copy
  float* scores;           // sweep 2 output
  int normalize;
  int bf16;                // operand type of Q and K: bf16 (1) or fp16 (0)
  int max_blocks;          // ceil(max_seqlen / kBlockRows)
  int n_items;             // (sequence, stationary block) pairs of one (layer, head)
  int total_items;         // n_items * n_layers * Hq
  int n_lh;                // n_layers * Hq
  int tail_lh;             // the last tail_lh (layer, head) pairs are handed out heaviest item first across all of them
  int* counter;            // work counter, zero at launch
  int32_t* status;
  int withhold_first_item; // diagnostic: the producer warp fetches its first item and then stops before announcing
                           // it or issuing any copy for it, so that every consumer's first wait runs out
};

template <int D>
struct PSmem {
  static constexpr int kTileBytes = kTile * D * 2;
  static constexpr int kBlockBytes = kTile * 128;
  static constexpr int kFixedOff = 0;                            // the stationary quarters
  static constexpr int kRingOff = kQ * kTileBytes;
  static constexpr int kAuxOff = kRingOff + kRing * kTileBytes;
  static constexpr int kAuxBytes = 26624;
  static constexpr int kTotal = kAuxOff + kAuxBytes + 1024;
};

struct PAux {
  unsigned long long full[kRing], empty[kRing];
  unsigned long long fixed_full, fixed_empty;
  unsigned long long acc_full[kQ], acc_empty[kQ];     // [quarter]
  unsigned long long item_full[2], item_empty[2];
  unsigned long long epi_bar;                         // all epilogue warps (sweep 2: a chunk of -lse2 is in place;
                                                      // sweep 1 with an observation window: slots merge)
  unsigned long long drain[kIssueWarps];
  uint32_t tmem_base;
  int abort_flag;
  int item[2][8];                                     // layer, head, seq, block, n_tiles (layer < 0: no more work)
  alignas(16) float lse_chunk[2][kLseChunk * kTile];  // [buffer][streamed tile inside the chunk][query]: minus lse2
  alignas(16) float part[2][kQ][2][kTile];            // [item parity][slot][max, sum][row]: sweep 1, replicated quarters
};

// Geometry of one work item, derived identically by every role.
template <bool kColsum>
struct Geo {
  int layer, h, hk, t0, L, blk, first_stream, n_iter;
  int ws;                      // first query row that votes (0 without an observation window)
  bool causal;
  int nq;                      // quarters of the block that hold rows of the sequence
  // The four accumulator slots normally hold the four quarters.  In sweep 1 with an observation window only the
  // quarters with voting queries have work; when these are one or two, each is loaded into rep = 4 or 2 slots and
  // slot s takes the streamed tiles it with it % rep == s % rep, so that all four epilogue groups stay busy.
  int rep, v0;                 // slots per voting quarter; first voting quarter
  __device__ __forceinline__ Geo(const Shape& s, const int* it) {
    layer = it[0]; h = it[1]; hk = h / s.G; blk = it[3];
    const int seq = it[2], n_tiles = it[4];
    t0 = __ldg(s.cu_seqlens + seq);
    L = __ldg(s.cu_seqlens + seq + 1) - t0;
    causal = s.causal != 0;
    nq = min(kQ, (L - blk * kBlockRows + kTile - 1) / kTile);
    ws = (s.window > 0 && L > s.window) ? L - s.window : 0;
    rep = 1; v0 = 0;
    if (kColsum) {                                                      // stationary keys, streamed query tiles
      first_stream = max(causal ? kQ * blk : 0, ws / kTile);
      n_iter = n_tiles - first_stream;
    } else {                                                            // stationary queries, streamed key tiles
      first_stream = 0;
      n_iter = causal ? min(kQ * blk + kQ, n_tiles) : n_tiles;
      if (ws > blk * kBlockRows) v0 = min(nq - 1, (ws - blk * kBlockRows) / kTile);
      if (s.window > 0) rep = nq - v0 == 1 ? 4 : (nq - v0 == 2 ? 2 : 1);
    }
  }
  __device__ __forceinline__ int n_slots() const { return rep > 1 ? kQ : nq; }
  __device__ __forceinline__ int quarter(int slot) const { return rep > 1 ? v0 + slot / rep : slot; }
  // does streamed tile `it` contribute to slot `sl` (causal: the quarter's own tile index is kQ*blk + quarter)
  __device__ __forceinline__ bool active(int sl, int it) const {
    const int qd = quarter(sl);
    if (qd >= nq || qd < v0) return false;                              // no rows, or no voting query
    if (rep > 1 && it % rep != sl % rep) return false;
    if (!causal) return true;
    return kColsum ? first_stream + it >= kQ * blk + qd : it <= kQ * blk + qd;
  }
  __device__ __forceinline__ bool diag(int sl, int it) const {
    const int qd = quarter(sl);
    return causal && (kColsum ? first_stream + it == kQ * blk + qd : it == kQ * blk + qd);
  }
};

// kPolls: polls of every bounded barrier wait (a compile-time constant: the epilogue has no register to spare for it).
template <int D, bool kColsum, uint32_t kPolls>
__global__ void __launch_bounds__(kThreads, 1)
score_persist_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                     const PersistArgs a) {
  using SL = PSmem<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  PAux* aux = reinterpret_cast<PAux*>(smem + SL::kAuxOff);
  volatile int* abort_flag = &aux->abort_flag;
  const uint32_t fixed_addr = smem_u32(smem + SL::kFixedOff);
  const uint32_t ring_addr = smem_u32(smem + SL::kRingOff);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const Shape& s = a.s;

  if (warp == 0) {
    if (lane == 0) {
      // a launch that already failed somewhere is not worth finishing
      aux->abort_flag = *reinterpret_cast<volatile int32_t*>(a.status) != 0;
      for (int i = 0; i < kRing; ++i) { mbar_init(smem_u32(&aux->full[i]), 1); mbar_init(smem_u32(&aux->empty[i]), kIssueWarps); }
      mbar_init(smem_u32(&aux->fixed_full), 1);
      mbar_init(smem_u32(&aux->fixed_empty), kIssueWarps);
      for (int i = 0; i < kIssueWarps; ++i) mbar_init(smem_u32(&aux->drain[i]), 1);
      for (int i = 0; i < kQ; ++i) {
        mbar_init(smem_u32(&aux->acc_full[i]), 1);
        mbar_init(smem_u32(&aux->acc_empty[i]), 4);
      }
      mbar_init(smem_u32(&aux->epi_bar), kEpiWarps);
      for (int i = 0; i < 2; ++i) {
        mbar_init(smem_u32(&aux->item_full[i]), 1);
        mbar_init(smem_u32(&aux->item_empty[i]), kIssueWarps + kEpiWarps);
      }
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
  const uint32_t tmem_base = aux->tmem_base;
  const bool dead = aux->abort_flag != 0;

  const CUtensorMap* map_fixed = kColsum ? &map_k : &map_q;
  const CUtensorMap* map_stream = kColsum ? &map_q : &map_k;

  if (dead) {
    // nothing to do
  } else if (warp == 0) {
    // ------------------------------ work fetch + TMA producer ------------------------------
    int n_item = 0, n_stream = 0;
    int issued_item = 0;              // lane 0: items whose stationary load was issued
    bool alive = true;
    while (alive) {
      const int slot = n_item & 1;
      int idx = 0;
      bool ok = true;
      if (lane == 0) {
        ok = mbar_wait(smem_u32(&aux->item_empty[slot]), ((n_item >> 1) & 1) ^ 1, abort_flag, kPolls);
        if (ok) idx = atomicAdd(a.counter, 1);
      }
      ok = __shfl_sync(0xFFFFFFFFu, (int)ok, 0) != 0;
      idx = __shfl_sync(0xFFFFFFFFu, idx, 0);
      if (!ok) break;
      if (idx >= a.total_items) {
        if (lane == 0) { aux->item[slot][0] = -1; mbar_arrive(smem_u32(&aux->item_full[slot])); }
        break;
      }
      if (a.withhold_first_item) break;        // nothing is in flight: the consumers' bounded waits end the CTA
      // (layer, head)-major order keeps the CTAs that run together on a few heads (their Q and K stay in L2); the
      // last pairs are taken weight-major instead, so that the launch does not end with a few CTAs on the heaviest
      // items of the last head while the others idle (a launch with few items is all tail)
      int lh, rank;
      const int head_part = (a.n_lh - a.tail_lh) * a.n_items;
      if (idx < head_part) {
        lh = idx / a.n_items; rank = idx - lh * a.n_items;
      } else {
        const int j = idx - head_part;
        rank = j / a.tail_lh; lh = a.n_lh - a.tail_lh + (j - rank * a.tail_lh);
      }
      int seq, blk, nblk;
      decode_item(s.cu_seqlens, s.n_seqs, a.max_blocks, rank, !kColsum, lane, seq, blk, nblk, kBlockRows, s.window);
      if (lane == 0) {
        int* it = aux->item[slot];
        it[0] = lh / s.Hq; it[1] = lh - it[0] * s.Hq; it[2] = seq; it[3] = blk;
        it[4] = (__ldg(s.cu_seqlens + seq + 1) - __ldg(s.cu_seqlens + seq) + kTile - 1) / kTile;
        mbar_arrive(smem_u32(&aux->item_full[slot]));
        const Geo<kColsum> g(s, it);
        const int head_fixed = kColsum ? g.hk : g.h, head_stream = kColsum ? g.h : g.hk;
        // the stationary buffer is free once every MMA of the previous item has retired
        ok = mbar_wait(smem_u32(&aux->fixed_empty), (n_item & 1) ^ 1, abort_flag, kPolls);
        if (ok) {
          const int n_slots = g.n_slots();
          mbar_expect_tx(smem_u32(&aux->fixed_full), n_slots * SL::kTileBytes);
          for (int sl = 0; sl < n_slots; ++sl)
#pragma unroll
            for (int kb = 0; kb < D / 64; ++kb)
              tma_load_4d(fixed_addr + sl * SL::kTileBytes + kb * SL::kBlockBytes, map_fixed, smem_u32(&aux->fixed_full),
                          kb * 64, g.t0 + g.blk * kBlockRows + g.quarter(sl) * kTile, head_fixed, g.layer);
          issued_item = n_item + 1;
          for (int i = 0; ok && i < g.n_iter; ++i, ++n_stream) {
            const int rs = n_stream % kRing;
            ok = mbar_wait(smem_u32(&aux->empty[rs]), ((n_stream / kRing) & 1) ^ 1, abort_flag, kPolls);
            if (!ok) break;
            mbar_expect_tx(smem_u32(&aux->full[rs]), SL::kTileBytes);
#pragma unroll
            for (int kb = 0; kb < D / 64; ++kb)
              tma_load_4d(ring_addr + rs * SL::kTileBytes + kb * SL::kBlockBytes, map_stream, smem_u32(&aux->full[rs]),
                          kb * 64, g.t0 + (g.first_stream + i) * kTile, head_stream, g.layer);
          }
        }
      }
      alive = __shfl_sync(0xFFFFFFFFu, (int)ok, 0) != 0;
      n_stream = __shfl_sync(0xFFFFFFFFu, n_stream, 0);
      ++n_item;
    }
    if (lane == 0 && *abort_flag) {
      // give the copies in flight a bounded time to land before the CTA's shared memory is released
      for (int q = max(0, n_stream - kRing); q < n_stream; ++q)
        for (uint32_t i = 0; i < kDrainPolls && !mbar_try_wait(smem_u32(&aux->full[q % kRing]), (q / kRing) & 1); ++i) {}
      if (issued_item > 0)
        for (uint32_t i = 0; i < kDrainPolls && !mbar_try_wait(smem_u32(&aux->fixed_full), (issued_item - 1) & 1); ++i) {}
    }
  } else if (warp <= kIssueWarps) {
    // ------------------------------ MMA issuers ------------------------------
    // One thread per pair of stationary quarters.  tcgen05.mma blocks its issuer while the tensor core's queue is
    // full, and the queue is short, so a lone issuer leaves the pipe idle whenever it has to poll a barrier; with
    // two issuers one polls while the other's instructions are queued.
    if (lane == 0) {
      const int iw = warp - 1;
      const uint32_t idesc = make_idesc(kTile, kTile, a.bf16 != 0);
      int n_item = 0, n_stream = 0, cnt[kQPerIssuer] = {};
      bool ok = true;
      while (ok) {
        const int slot = n_item & 1;
        ok = mbar_wait(smem_u32(&aux->item_full[slot]), (n_item >> 1) & 1, abort_flag, kPolls);
        if (!ok) break;
        int it[5];
#pragma unroll
        for (int i = 0; i < 5; ++i) it[i] = aux->item[slot][i];
        mbar_arrive(smem_u32(&aux->item_empty[slot]));
        if (it[0] < 0) break;
        const Geo<kColsum> g(s, it);
        ok = mbar_wait(smem_u32(&aux->fixed_full), n_item & 1, abort_flag, kPolls);
        for (int i = 0; ok && i < g.n_iter; ++i, ++n_stream) {
          const int rs = n_stream % kRing;
          // also when its quarters skip the tile: the wait keeps the issuer from running a whole ring ahead of
          // the other one, whose arrival on empty[rs] must fall into the same phase as this one's
          ok = mbar_wait(smem_u32(&aux->full[rs]), (n_stream / kRing) & 1, abort_flag, kPolls);
          if (!ok) break;
#pragma unroll
          for (int u = 0; u < kQPerIssuer; ++u) {
            if (!ok) break;
            const int qd = kQPerIssuer * iw + u;
            if (!g.active(qd, i)) continue;
            const int c = cnt[u]++;                 // the quarter's accumulator is reused every time: phase c & 1
            ok = mbar_wait(smem_u32(&aux->acc_empty[qd]), (c & 1) ^ 1, abort_flag, kPolls);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + qd * kTile;
#pragma unroll
            for (int k = 0; k < D / 16; ++k) {
              const uint32_t off = (k >> 2) * SL::kBlockBytes + (k & 3) * 32;
              umma_bf16(d_tmem, smem_desc_sw128(fixed_addr + qd * SL::kTileBytes + off),
                        smem_desc_sw128(ring_addr + rs * SL::kTileBytes + off), idesc, k > 0);
            }
            umma_commit(smem_u32(&aux->acc_full[qd]));
          }
          if (!ok) break;
          // this issuer is done with the ring slot (a commit with nothing pending arrives at once)
          umma_commit(smem_u32(&aux->empty[rs]));
        }
        if (!ok) break;
        umma_commit(smem_u32(&aux->fixed_empty));
        ++n_item;
      }
      if (*abort_flag) {
        // wait (bounded) until every MMA already issued has retired before TMEM and shared memory go away
        umma_commit(smem_u32(&aux->drain[iw]));
        for (uint32_t i = 0; i < kDrainPolls && !mbar_try_wait(smem_u32(&aux->drain[iw]), 0); ++i) {}
      }
    }
  } else {
    // ------------------------------ epilogue groups ------------------------------
    const int gi = (warp - 1 - kIssueWarps) >> 2;  // group = stationary quarter; it owns that quarter's accumulator
    const int quarter = warp & 3;                  // TMEM lanes this warp may read
    const int r = quarter * 32 + lane;             // row of the accumulator = TMEM lane = index inside the group
    const uint32_t t_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + gi * kTile;
    const uint32_t acc_full = smem_u32(&aux->acc_full[gi]), acc_empty = smem_u32(&aux->acc_empty[gi]);
    const float scale = a.scale_log2;
    const f32x2 scale2 = splat2(scale);
    const float ninf = __int_as_float(0xFF800000);
    int n_item = 0, cnt = 0, n_esync = 0;
    bool ok = true;

    // barrier among all 16 epilogue warps; bounded like every other wait
    auto epi_sync = [&]() {
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&aux->epi_bar));
      ok = mbar_wait(smem_u32(&aux->epi_bar), n_esync & 1, abort_flag, kPolls) && ok;
      ++n_esync;
    };
    auto release = [&]() {                         // accumulator drained: hand it back to its issuer
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty);
    };

    while (true) {
      const int slot = n_item & 1;
      ok = mbar_wait(smem_u32(&aux->item_full[slot]), (n_item >> 1) & 1, abort_flag, kPolls) && ok;
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      int it[5];
#pragma unroll
      for (int i = 0; i < 5; ++i) it[i] = aux->item[slot][i];
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&aux->item_empty[slot]));
      if (it[0] < 0) break;
      const Geo<kColsum> g(s, it);
      const int row = g.blk * kBlockRows + g.quarter(gi) * kTile + r;   // token of this thread inside the sequence
      const size_t out = ((size_t)g.layer * s.Hq + g.h) * s.T + g.t0 + row;

      if constexpr (kColsum) {
        const float* lse_row = a.lse + ((size_t)g.layer * s.Hq + g.h) * s.T + g.t0;
        // Minus lse2 of the streamed queries reaches the epilogue threads through shared memory, kLseChunk tiles
        // at a time and once for all four groups: all 16 warps fill the next chunk's buffer, then work through the
        // current chunk, and meet once per chunk (the buffer of chunk k is rewritten as chunk k + 2 only after
        // everybody left chunk k).
        const int et = tid - 32 * (1 + kIssueWarps);
        auto fill = [&](int k) {
          float* dst = aux->lse_chunk[k & 1];
#pragma unroll
          for (int e = et; e < kLseChunk * kTile; e += kEpiWarps * 32) {
            const int i = kLseChunk * k + (e >> 7);
            const int j = (g.first_stream + i) * kTile + (e & (kTile - 1));
            dst[e] = (i < g.n_iter && j < g.L && j >= g.ws) ? -(__ldg(lse_row + j) * a.lse_mul) : ninf;
          }
        };
        f32x2 acc[2] = {0ull, 0ull};
        const int n_chunks = (g.n_iter + kLseChunk - 1) / kLseChunk;
        fill(0);
        epi_sync();
        for (int k = 0; k < n_chunks && ok; ++k) {
          if (k + 1 < n_chunks) fill(k + 1);
          const int i_end = min(g.n_iter, kLseChunk * (k + 1));
          for (int i = kLseChunk * k; i < i_end && ok; ++i) {
            if (!g.active(gi, i)) continue;
            const int c = cnt++;
            const float* lse_buf = aux->lse_chunk[k & 1] + (i & (kLseChunk - 1)) * kTile;
            ok = mbar_wait(acc_full, c & 1, abort_flag, kPolls) && ok;
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            if (g.diag(gi, i))
              sweep_tile<true>(t_acc, [&](const uint32_t (&v)[16], int p) { colsum_piece<true>(v, lse_buf + p * 16, scale2, r, p * 16, acc); }, release);
            else
              sweep_tile(t_acc, [&](const uint32_t (&v)[16], int p) { colsum_piece<false>(v, lse_buf + p * 16, scale2, r, p * 16, acc); }, release);
          }
          epi_sync();
        }
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
        float total = sum4(acc);
        if (row < g.L) {
          if (a.normalize) total = total / (float)(g.L - g.ws);
          a.scores[out] = total;
        }
      } else {
        float m = __int_as_float(0xFF800000);                   // running max (log2 domain) of this row
        f32x2 sum2[2] = {0ull, 0ull};                           // packed partial sums of 2^(x - m)
        for (int i = 0; i < g.n_iter && ok; ++i) {
          if (!g.active(gi, i)) continue;
          const int c = cnt++;
          ok = mbar_wait(acc_full, c & 1, abort_flag, kPolls) && ok;
          ok = __all_sync(0xFFFFFFFFu, ok);
          if (!ok) break;
          tc_fence_after();
          // keys of this tile that count for this row: up to the diagonal (causal) and inside the sequence
          const int n_valid = g.causal ? (g.diag(gi, i) ? r + 1 : kTile) : min(kTile, g.L - i * kTile);
          // masked columns, or a row that has no reference yet (its first tile): exact maxima, piece by piece
          if (__any_sync(0xFFFFFFFFu, n_valid < kTile || !(m > -3.0e38f)))
            sweep_tile<true>(t_acc, [&](const uint32_t (&v)[16], int p) { lse_piece<true>(v, scale, scale2, n_valid - p * 16, m, sum2); }, release);
          else
            lse_tile_lazy(t_acc, scale, scale2, m, sum2, release);
        }
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
        float sum = sum4(sum2);
        if (s.window > 0) {                  // slots that share a quarter merge their (max, sum) through shared memory
          float* pm = aux->part[n_item & 1][gi][0];
          float* ps = aux->part[n_item & 1][gi][1];
          pm[r] = m;
          ps[r] = sum;
          epi_sync();
          ok = __all_sync(0xFFFFFFFFu, ok);
          if (!ok) break;
          if (g.rep > 1 && gi % g.rep == 0) {
            float big = m;
            for (int u = 1; u < g.rep; ++u) big = fmaxf(big, aux->part[n_item & 1][gi + u][0][r]);
            float tot = sum > 0.f ? sum * ex2(m - big) : 0.f;
            for (int u = 1; u < g.rep; ++u) {
              const float mu = aux->part[n_item & 1][gi + u][0][r], su = aux->part[n_item & 1][gi + u][1][r];
              tot += su > 0.f ? su * ex2(mu - big) : 0.f;
            }
            m = big;
            sum = tot;
          }
        }
        if (row < g.L && row >= g.ws && (g.rep == 1 || gi % g.rep == 0)) {
          const float lse2 = m + log2f(sum);
          a.lse2_out[out] = lse2;
          if (a.lse_nat_out) a.lse_nat_out[out] = lse2 * 0.69314718055994530942f;
        }
      }
      ++n_item;
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

template <int D, bool kColsum, uint32_t kPolls>
int launch_persist_polls(const CUtensorMap& mq, const CUtensorMap& mk, const PersistArgs& a, int n_sms, cudaStream_t stream) {
  auto kern = score_persist_kernel<D, kColsum, kPolls>;
  constexpr int smem = PSmem<D>::kTotal;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return KVCRUSH_ERR_CUDA;
  const int blocks = a.total_items < n_sms ? a.total_items : n_sms;
  kern<<<(unsigned)blocks, kThreads, smem, stream>>>(mq, mk, a);
  return check_launch();
}

template <int D, bool kColsum>
int launch_persist(const CUtensorMap& mq, const CUtensorMap& mk, const PersistArgs& a, bool short_waits, int n_sms,
                   cudaStream_t stream) {
  return short_waits ? launch_persist_polls<D, kColsum, kShortWaitPolls>(mq, mk, a, n_sms, stream)
                     : launch_persist_polls<D, kColsum, kWaitPolls>(mq, mk, a, n_sms, stream);
}

}  // namespace

size_t score_tensor_counter_bytes() { return 256; }

int score_tensor_plan(const Shape& s, const TensorView& Q, const TensorView& K, ScoreTensorMaps* maps) {
  static_assert(sizeof(CUtensorMap) == sizeof(maps->q) && alignof(CUtensorMap) <= 64, "tensor map storage");
  if (Q.dtype != K.dtype || (Q.dtype != KVCRUSH_BF16 && Q.dtype != KVCRUSH_FP16)) return TENSOR_PLAN_NO;
  if (s.D < 8 || s.D > 128 || s.D % 8 != 0) return TENSOR_PLAN_NO;      // other widths ride in the 64- or 128-wide kernel
  if (s.T < 1) return TENSOR_PLAN_NO;
  if (encode_fn() == nullptr) return TENSOR_PLAN_NO_ENCODER;
  if (!make_map(reinterpret_cast<CUtensorMap*>(maps->q), Q, s.D, s.T, s.Hq, s.n_layers) ||
      !make_map(reinterpret_cast<CUtensorMap*>(maps->k), K, s.D, s.T, s.Hkv, s.n_layers))
    return TENSOR_PLAN_NO;                                               // strides or extents the TMA unit cannot take
  return TENSOR_PLAN_OK;
}


int launch_score_tensor(const Shape& s, const int32_t* cu_host, const TensorView& Q, const ScoreTensorMaps& maps,
                        float scale_log2, const float* lse_in, float lse_in_mul, float* lse2_ws,
                        int* counters, float* scores, float* lse_out, int normalize, int32_t* status,
                        const ScoreDiag& diag, cudaStream_t stream) {
  static_assert(sizeof(PAux) <= 26624, "aux block too large");
  if (!(scale_log2 > 0.f)) return KVCRUSH_ERR_UNSUPPORTED;
  const CUtensorMap& mq = *reinterpret_cast<const CUtensorMap*>(maps.q);
  const CUtensorMap& mk = *reinterpret_cast<const CUtensorMap*>(maps.k);
  int dev = 0, n_sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n_sms < 1)
    return KVCRUSH_ERR_CUDA;
  PersistArgs a{};
  a.s = s; a.scale_log2 = scale_log2; a.normalize = normalize; a.bf16 = Q.dtype == KVCRUSH_BF16; a.status = status; a.scores = scores;
  const bool sw = diag.short_waits != 0;
  a.withhold_first_item = diag.withhold_first_item;
  a.max_blocks = (s.max_seqlen + kBlockRows - 1) / kBlockRows;
  // work items per (layer, head): every 512-row block for the column sweep; for the row sweep only the
  // blocks that hold voting queries
  long long items_col = 0, items_row = 0;
  for (int i = 0; i < s.n_seqs; ++i) {
    const int len = cu_host[i + 1] - cu_host[i];
    const int nb = (len + kBlockRows - 1) / kBlockRows;
    const int first = (s.window > 0 && len > s.window) ? (len - s.window) / kBlockRows : 0;
    items_col += nb;
    items_row += nb - first;
  }
  if (items_col == 0) return KVCRUSH_OK;
  if (items_col * s.n_layers * s.Hq > 0x7FFFFFFFLL) return KVCRUSH_ERR_UNSUPPORTED;
  if (cudaMemsetAsync(counters, 0, 2 * sizeof(int), stream) != cudaSuccess) return KVCRUSH_ERR_CUDA;
  a.n_lh = s.n_layers * s.Hq;
  auto tail_pairs = [&](long long items) {       // pairs whose items make up about four rounds of the grid
    const long long t = (4LL * n_sms + items - 1) / items;
    return (int)(t < a.n_lh ? t : a.n_lh);
  };
  int rc;
  if (!lse_in) {
    a.lse2_out = lse2_ws; a.lse_nat_out = lse_out; a.counter = counters;
    a.n_items = (int)items_row; a.total_items = (int)(items_row * s.n_layers * s.Hq);
    a.tail_lh = tail_pairs(items_row);
    rc = s.D > 64 ? launch_persist<128, false>(mq, mk, a, sw, n_sms, stream) : launch_persist<64, false>(mq, mk, a, sw, n_sms, stream);
    if (rc != KVCRUSH_OK) return rc;
    a.lse = lse2_ws; a.lse_mul = 1.f;
  } else {
    a.lse = lse_in; a.lse_mul = lse_in_mul;
  }
  a.counter = counters + 1;
  a.n_items = (int)items_col; a.total_items = (int)(items_col * s.n_layers * s.Hq);
  a.tail_lh = tail_pairs(items_col);
  return s.D > 64 ? launch_persist<128, true>(mq, mk, a, sw, n_sms, stream) : launch_persist<64, true>(mq, mk, a, sw, n_sms, stream);
}

}  // namespace kvc
