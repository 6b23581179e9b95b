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
constexpr uint32_t kSpinLimit = 1u << 20;

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the wait ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 31u) == 31u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void named_bar_sync(int id, int n) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory");
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 2^x on the FMA pipe for x <= ~0 (any magnitude): round-to-nearest split x = n + f, f in [-0.5, 0.5],
// cubic minimax polynomial for 2^f (relative error 7.5e-5), exponent bits of n added to the result.
// The special-function unit delivers 16 ex2 per clock per SM and is the busiest unit of both sweeps;
// sending a fixed share of the exponentials down this path takes load off it.
__device__ __forceinline__ float exp2_poly(float x) {
  x = fmaxf(x, -125.f);                              // keeps the result a normal number (also maps -inf)
  const float t = x + 12582912.f;                    // 1.5 * 2^23: the integer part lands in the low mantissa bits
  const float f = x - (t - 12582912.f);
  float p = fmaf(f, 0.0551716648f, 0.2426111251f);
  p = fmaf(p, f, 0.6932609677f);
  p = fmaf(p, f, 0.9999280572f);
  return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
}

#ifndef KVC_POLY_PER8
#define KVC_POLY_PER8 2                              // of every 8 exponentials, this many use exp2_poly
#endif
__host__ __device__ constexpr bool poly_slot(int i) {
  return ((i % 8 + 1) * KVC_POLY_PER8) / 8 > ((i % 8) * KVC_POLY_PER8) / 8;
}
template <int I>
__device__ __forceinline__ float exp2_mix(float x) {
  if constexpr (poly_slot(I)) return exp2_poly(x); else return ex2(x);
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// 16 consecutive fp32 columns of this thread's TMEM lane (asynchronous: see tmem_wait16)
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}
// Waits for every TMEM load of this thread.  The registers are listed as read-write operands so that
// no use of them can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_wait16(uint32_t (&v)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                 "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15])
               :: "memory");
}

// Streams the 128 columns of one accumulator through two 16-column register buffers: the load of the next
// piece is in flight while the current one is processed.  `release` runs once the last load has landed.
template <class Piece, class Release>
__device__ __forceinline__ void sweep_tile(uint32_t taddr, Piece&& piece, Release&& release) {
  uint32_t va[16], vb[16];
  tmem_ld16(taddr, va);
  tmem_wait16(va);
#pragma unroll
  for (int p = 0; p < 8; p += 2) {
    tmem_ld16(taddr + (p + 1) * 16, vb);
    piece(va, p);
    tmem_wait16(vb);
    if (p == 6) release();
    if (p < 6) tmem_ld16(taddr + (p + 2) * 16, va);
    piece(vb, p + 1);
    if (p < 6) tmem_wait16(va);
  }
}

// ---- sweep 2: 16 columns (queries) of this thread's key row -------------------------------------
template <bool kDiag>
__device__ __forceinline__ void colsum_piece(const uint32_t (&v)[16], const float* lse16, float scale, int r, int c0,
                                             float (&acc)[4]) {
  const float4* l4 = reinterpret_cast<const float4*>(lse16);
#pragma unroll
  for (int c4 = 0; c4 < 4; ++c4) {
    const float4 l = l4[c4];
    float e0, e1, e2, e3;
    if (c4 == 0) {
      e0 = exp2_mix<0>(fmaf(__uint_as_float(v[0]), scale, -l.x)); e1 = exp2_mix<1>(fmaf(__uint_as_float(v[1]), scale, -l.y));
      e2 = exp2_mix<2>(fmaf(__uint_as_float(v[2]), scale, -l.z)); e3 = exp2_mix<3>(fmaf(__uint_as_float(v[3]), scale, -l.w));
    } else if (c4 == 1) {
      e0 = exp2_mix<4>(fmaf(__uint_as_float(v[4]), scale, -l.x)); e1 = exp2_mix<5>(fmaf(__uint_as_float(v[5]), scale, -l.y));
      e2 = exp2_mix<6>(fmaf(__uint_as_float(v[6]), scale, -l.z)); e3 = exp2_mix<7>(fmaf(__uint_as_float(v[7]), scale, -l.w));
    } else if (c4 == 2) {
      e0 = exp2_mix<0>(fmaf(__uint_as_float(v[8]), scale, -l.x)); e1 = exp2_mix<1>(fmaf(__uint_as_float(v[9]), scale, -l.y));
      e2 = exp2_mix<2>(fmaf(__uint_as_float(v[10]), scale, -l.z)); e3 = exp2_mix<3>(fmaf(__uint_as_float(v[11]), scale, -l.w));
    } else {
      e0 = exp2_mix<4>(fmaf(__uint_as_float(v[12]), scale, -l.x)); e1 = exp2_mix<5>(fmaf(__uint_as_float(v[13]), scale, -l.y));
      e2 = exp2_mix<6>(fmaf(__uint_as_float(v[14]), scale, -l.z)); e3 = exp2_mix<7>(fmaf(__uint_as_float(v[15]), scale, -l.w));
    }
    if constexpr (kDiag) {                          // causal: the query (column) must not precede the key (row)
      const int c = c0 + 4 * c4;
      e0 = c + 0 >= r ? e0 : 0.f; e1 = c + 1 >= r ? e1 : 0.f;
      e2 = c + 2 >= r ? e2 : 0.f; e3 = c + 3 >= r ? e3 : 0.f;
    }
    acc[0] += e0; acc[1] += e1; acc[2] += e2; acc[3] += e3;
  }
}

// ---- sweep 1: 16 columns (keys) of this thread's query row; online max / sum in the log2 domain ----
template <bool kMasked>
__device__ __forceinline__ void lse_piece(const uint32_t (&v)[16], float scale, int c_lim, float& m, float& sum) {
  float x[16];
#pragma unroll
  for (int c = 0; c < 16; ++c) x[c] = __uint_as_float(v[c]);
  if constexpr (kMasked) {
    if (c_lim <= 0) return;                         // nothing of this piece belongs to the row
#pragma unroll
    for (int c = 0; c < 16; ++c) x[c] = c < c_lim ? x[c] : __int_as_float(0xFF800000);
  }
  const float m0 = max3(x[0], x[1], x[2]), m1 = max3(x[3], x[4], x[5]), m2 = max3(x[6], x[7], x[8]);
  const float m3 = max3(x[9], x[10], x[11]), m4 = max3(x[12], x[13], x[14]);
  const float cmax = fmaxf(max3(m0, m1, m2), max3(m3, m4, x[15]));
  const float m_new = fmaxf(m, cmax * scale);
  if (m_new > m) { sum *= ex2(m - m_new); m = m_new; }
  float s0, s1, s2, s3;
  s0 = exp2_mix<0>(fmaf(x[0], scale, -m)); s1 = exp2_mix<1>(fmaf(x[1], scale, -m));
  s2 = exp2_mix<2>(fmaf(x[2], scale, -m)); s3 = exp2_mix<3>(fmaf(x[3], scale, -m));
  s0 += exp2_mix<4>(fmaf(x[4], scale, -m)); s1 += exp2_mix<5>(fmaf(x[5], scale, -m));
  s2 += exp2_mix<6>(fmaf(x[6], scale, -m)); s3 += exp2_mix<7>(fmaf(x[7], scale, -m));
  s0 += exp2_mix<0>(fmaf(x[8], scale, -m)); s1 += exp2_mix<1>(fmaf(x[9], scale, -m));
  s2 += exp2_mix<2>(fmaf(x[10], scale, -m)); s3 += exp2_mix<3>(fmaf(x[11], scale, -m));
  s0 += exp2_mix<4>(fmaf(x[12], scale, -m)); s1 += exp2_mix<5>(fmaf(x[13], scale, -m));
  s2 += exp2_mix<6>(fmaf(x[14], scale, -m)); s3 += exp2_mix<7>(fmaf(x[15], scale, -m));
  sum += (s0 + s1) + (s2 + s3);
}

// Shared-memory matrix descriptor of a K-major tile stored as 128-byte rows with the 128B swizzle
// (rows of 64 bf16; 8-row groups 1024 bytes apart).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);          // start address
  d |= (uint64_t)1 << 16;                           // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024u >> 4) << 32;                // stride byte offset: 8 rows * 128 B
  d |= (uint64_t)1 << 46;                           // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                           // 128-byte swizzle
  return d;
}

// kind::f16 instruction descriptor: fp32 accumulate, bf16 x bf16, both operands K-major, M x N.
__host__ __device__ constexpr uint32_t make_idesc(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ------------------------------------------------------------------------------------------------
// work decomposition: rank -> (sequence, tile), heaviest first
// ------------------------------------------------------------------------------------------------
// Items are (sequence, tile) pairs; an item's weight w is the number of 128x128 tiles it sweeps
// (causal: query tile q sweeps q+1 key tiles; key tile k sweeps n-k query tiles).  Rank j counts items
// in order of decreasing w, sequences in order inside one w.  Runs on one full warp.
__device__ __forceinline__ void decode_item(const int32_t* __restrict__ cu, int n_seqs, int max_tiles, int j,
                                            bool row_sweep, int lane, int& seq, int& tile, int& n_tiles) {
  int rem = j;
  seq = 0; tile = 0; n_tiles = 0;
  for (int w = max_tiles; w >= 1; --w) {
    for (int base = 0; base < n_seqs; base += 32) {
      const int s = base + lane;
      const int nt = s < n_seqs ? (__ldg(cu + s + 1) - __ldg(cu + s) + kTile - 1) / kTile : 0;
      const unsigned mask = __ballot_sync(0xFFFFFFFFu, nt >= w);
      const int cnt = __popc(mask);
      if (rem < cnt) {
        const int pos = __fns(mask, 0, rem + 1);
        seq = base + pos;
        n_tiles = __shfl_sync(0xFFFFFFFFu, nt, pos);
        tile = row_sweep ? w - 1 : n_tiles - w;
        return;
      }
      rem -= cnt;
    }
  }
}

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
    bool ok = true;

    if constexpr (kColsum) {
      const float* lse_row = a.lse + ((size_t)layer * s.Hq + h) * s.T + t0;
      const float inf = __int_as_float(0x7F800000);
      auto load_lse = [&](int it) {                 // lse2 of this thread's query of streamed tile `it` (+inf past the end)
        const int j = (first_stream + it) * kTile + gtid;
        return (it < n_iter && j < L) ? __ldg(lse_row + j) * a.lse_mul : inf;
      };
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
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
          sweep_tile(t_acc, [&](const uint32_t (&v)[16], int p) { colsum_piece<true>(v, lse_buf + p * 16, scale, r, p * 16, acc); }, release);
        else
          sweep_tile(t_acc, [&](const uint32_t (&v)[16], int p) { colsum_piece<false>(v, lse_buf + p * 16, scale, r, p * 16, acc); }, release);
      }
      float total = (acc[0] + acc[1]) + (acc[2] + acc[3]);
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
      float m = __int_as_float(0xFF800000), sum = 0.f;        // running max (log2 domain) and sum of this row
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
          sweep_tile(t_acc, [&](const uint32_t (&v)[16], int p) { lse_piece<true>(v, scale, n_valid - p * 16, m, sum); }, release);
        else
          sweep_tile(t_acc, [&](const uint32_t (&v)[16], int p) { lse_piece<false>(v, scale, 16, m, sum); }, release);
      }
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
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// 4-D view (channel, token, head, layer) of a token-major bf16 tensor; box = 64 channels x 128 tokens.
bool make_map(CUtensorMap* map, const TensorView& t, int D, int T, int H, int n_layers) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  const cuuint64_t gdim[4] = {(cuuint64_t)D, (cuuint64_t)T, (cuuint64_t)H, (cuuint64_t)n_layers};
  auto stride_bytes = [](long long st) { return (cuuint64_t)(st > 0 ? st * 2 : 16); };
  const cuuint64_t gstride[3] = {stride_bytes(t.st), stride_bytes(t.sh), stride_bytes(t.sl)};
  const cuuint32_t box[4] = {64, (cuuint32_t)kTile, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(t.ptr), gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

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
