// Inline-PTX wrappers and per-element math shared by the tensor-core score kernels (tcgen05, TMEM, TMA,
// mbarrier), sm_100a only.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"

namespace kvc {
namespace tc {

constexpr uint32_t kSpinLimit = 1u << 20;        // polls of one bounded barrier wait

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
                                            bool row_sweep, int lane, int& seq, int& tile, int& n_tiles,
                                            int rows_per_item = 128) {
  int rem = j;
  seq = 0; tile = 0; n_tiles = 0;
  for (int w = max_tiles; w >= 1; --w) {
    for (int base = 0; base < n_seqs; base += 32) {
      const int s = base + lane;
      const int nt = s < n_seqs ? (__ldg(cu + s + 1) - __ldg(cu + s) + rows_per_item - 1) / rows_per_item : 0;
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


// ------------------------------------------------------------------------------------------------
// host side: tensor maps
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
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
inline bool make_map(CUtensorMap* map, const TensorView& t, int D, int T, int H, int n_layers) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  const cuuint64_t gdim[4] = {(cuuint64_t)D, (cuuint64_t)T, (cuuint64_t)H, (cuuint64_t)n_layers};
  auto stride_bytes = [](long long st) { return (cuuint64_t)(st > 0 ? st * 2 : 16); };
  const cuuint64_t gstride[3] = {stride_bytes(t.st), stride_bytes(t.sh), stride_bytes(t.sl)};
  const cuuint32_t box[4] = {64, 128u, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(t.ptr), gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


}  // namespace tc
}  // namespace kvc
