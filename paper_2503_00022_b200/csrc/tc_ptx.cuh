// Inline-PTX wrappers and per-element math shared by the tensor-core score kernels (tcgen05, TMEM, TMA,
// mbarrier), sm_100a only.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "common.cuh"

namespace kvc {
namespace tc {

constexpr uint32_t kWaitPolls = 1u << 20;        // polls of one bounded barrier wait
constexpr uint32_t kShortWaitPolls = 1u << 12;   // the same in the diagnostic build of the kernels (waits made to run out)
constexpr uint32_t kDrainPolls = 1u << 20;       // polls granted to copies and MMAs in flight after a role gave up; never shortened

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
// Bounded wait of at most `polls` polls.  Returns false when the wait ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t polls) {
  for (uint32_t i = 0; i < polls; ++i) {
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

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---- packed fp32x2 arithmetic (two floats in one 64-bit register, one instruction for both) ---------
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(uint32_t lo, uint32_t hi) {
  f32x2 d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
  return d;
}
__device__ __forceinline__ f32x2 pack2f(float lo, float hi) { return pack2(__float_as_uint(lo), __float_as_uint(hi)); }
__device__ __forceinline__ f32x2 splat2(float x) { return pack2f(x, x); }
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
  uint32_t a, b;
  asm("mov.b64 {%0, %1}, %2;" : "=r"(a), "=r"(b) : "l"(v));
  lo = __uint_as_float(a);
  hi = __uint_as_float(b);
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// 2^x for a pair on the special-function unit.
__device__ __forceinline__ f32x2 exp2_sfu2(f32x2 x) {
  float a, b;
  unpack2(x, a, b);
  return pack2f(ex2(a), ex2(b));
}
// 2^x for a pair on the FMA pipe, x <= ~0 (any magnitude): round-to-nearest split x = n + f, f in [-0.5, 0.5],
// cubic minimax polynomial for 2^f (relative error 7.5e-5), exponent bits of n added to the result.
// The special-function unit delivers 16 ex2 per clock per SM and is the busiest unit of both sweeps; a
// share of the exponentials can go down this path instead, at 6 packed + 6 scalar instructions a pair.
__device__ __forceinline__ f32x2 exp2_poly2(f32x2 x) {
  float x0, x1;
  unpack2(x, x0, x1);
  x = pack2f(fmaxf(x0, -125.f), fmaxf(x1, -125.f));           // keeps the result a normal number (also maps -inf)
  const f32x2 t = add2(x, splat2(12582912.f));                // 1.5 * 2^23: the integer part lands in the low mantissa bits
  const f32x2 n = add2(t, splat2(-12582912.f));
  const f32x2 f = fma2(n, splat2(-1.f), x);
  f32x2 p = fma2(f, splat2(0.0551716648f), splat2(0.2426111251f));
  p = fma2(p, f, splat2(0.6932609677f));
  p = fma2(p, f, splat2(0.9999280572f));
  float p0, p1, t0, t1;
  unpack2(p, p0, p1);
  unpack2(t, t0, t1);
  return pack2(__float_as_uint(p0) + (__float_as_uint(t0) << 23), __float_as_uint(p1) + (__float_as_uint(t1) << 23));
}

// Share of the exponentials that takes the FMA-pipe path, in pairs out of every 8 pairs (one 16-column piece), per sweep.
// Measured at the board power limit (32 layers x 32 heads x 8192 tokens, loops of several seconds): two pairs in
// eight are the best share for both sweeps; none costs cycles (the special-function unit saturates), two cost more
// instructions and energy than they save.
#ifndef KVC_POLY_PAIRS_LSE
#define KVC_POLY_PAIRS_LSE 2
#endif
#ifndef KVC_POLY_PAIRS_COLSUM
#define KVC_POLY_PAIRS_COLSUM 2
#endif
template <int J, int P>
__device__ __forceinline__ f32x2 exp2_mix2(f32x2 x) {
  constexpr bool poly = ((J % 8 + 1) * P) / 8 > ((J % 8) * P) / 8;
  if constexpr (poly) return exp2_poly2(x); else return exp2_sfu2(x);
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
// kRolled keeps the loop rolled (two pieces per iteration): for the tile kinds that are rare (diagonal and first
// tiles), so that their code does not push the common kind out of the instruction cache.
template <bool kRolled = false, class Piece, class Release>
__device__ __forceinline__ void sweep_tile(uint32_t taddr, Piece&& piece, Release&& release) {
  uint32_t va[16], vb[16];
  tmem_ld16(taddr, va);
  tmem_wait16(va);
  if constexpr (kRolled) {
#pragma unroll 1
    for (int p = 0; p < 8; p += 2) {
      tmem_ld16(taddr + (p + 1) * 16, vb);
      piece(va, p);
      tmem_wait16(vb);
      if (p == 6) release();
      if (p < 6) tmem_ld16(taddr + (p + 2) * 16, va);
      piece(vb, p + 1);
      if (p < 6) tmem_wait16(va);
    }
  } else {
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
}

// ---- sweep 2: 16 columns (queries) of this thread's key row -------------------------------------
// nlse16: MINUS the log2-domain row log-sum-exp of the 16 queries (-inf past the end of the sequence).
template <int J, bool kDiag>
__device__ __forceinline__ f32x2 colsum_pair(uint32_t v0, uint32_t v1, float nl0, float nl1, f32x2 scale2, int r, int c) {
  f32x2 e = exp2_mix2<J, KVC_POLY_PAIRS_COLSUM>(fma2(pack2(v0, v1), scale2, pack2f(nl0, nl1)));
  if constexpr (kDiag) {                            // causal: the query (column) must not precede the key (row)
    float e0, e1;
    unpack2(e, e0, e1);
    e = pack2f(c >= r ? e0 : 0.f, c + 1 >= r ? e1 : 0.f);
  }
  return e;
}
template <bool kDiag>
__device__ __forceinline__ void colsum_piece(const uint32_t (&v)[16], const float* nlse16, f32x2 scale2, int r, int c0,
                                             f32x2 (&acc)[2]) {
  const float4* l4 = reinterpret_cast<const float4*>(nlse16);
  const float4 la = l4[0], lb = l4[1], lc = l4[2], ld = l4[3];
  acc[0] = add2(acc[0], colsum_pair<0, kDiag>(v[0], v[1], la.x, la.y, scale2, r, c0 + 0));
  acc[1] = add2(acc[1], colsum_pair<1, kDiag>(v[2], v[3], la.z, la.w, scale2, r, c0 + 2));
  acc[0] = add2(acc[0], colsum_pair<2, kDiag>(v[4], v[5], lb.x, lb.y, scale2, r, c0 + 4));
  acc[1] = add2(acc[1], colsum_pair<3, kDiag>(v[6], v[7], lb.z, lb.w, scale2, r, c0 + 6));
  acc[0] = add2(acc[0], colsum_pair<4, kDiag>(v[8], v[9], lc.x, lc.y, scale2, r, c0 + 8));
  acc[1] = add2(acc[1], colsum_pair<5, kDiag>(v[10], v[11], lc.z, lc.w, scale2, r, c0 + 10));
  acc[0] = add2(acc[0], colsum_pair<6, kDiag>(v[12], v[13], ld.x, ld.y, scale2, r, c0 + 12));
  acc[1] = add2(acc[1], colsum_pair<7, kDiag>(v[14], v[15], ld.z, ld.w, scale2, r, c0 + 14));
}

// ---- sweep 1: 16 columns (keys) of this thread's query row; online max / sum in the log2 domain ----
// m: running maximum; sum2: two packed partial sums of 2^(x - m) (four floats to add up at the end).
template <bool kMasked>
__device__ __forceinline__ void lse_piece(const uint32_t (&v)[16], float scale, f32x2 scale2, int c_lim, float& m,
                                          f32x2 (&sum2)[2]) {
  uint32_t x[16];
#pragma unroll
  for (int c = 0; c < 16; ++c) x[c] = v[c];
  if constexpr (kMasked) {
    if (c_lim <= 0) return;                         // nothing of this piece belongs to the row
#pragma unroll
    for (int c = 0; c < 16; ++c) x[c] = c < c_lim ? x[c] : 0xFF800000u;
  }
#define KVC_F(i) __uint_as_float(x[i])
  const float m0 = max3(KVC_F(0), KVC_F(1), KVC_F(2)), m1 = max3(KVC_F(3), KVC_F(4), KVC_F(5));
  const float m2 = max3(KVC_F(6), KVC_F(7), KVC_F(8)), m3 = max3(KVC_F(9), KVC_F(10), KVC_F(11));
  const float m4 = max3(KVC_F(12), KVC_F(13), KVC_F(14));
  const float cmax = fmaxf(max3(m0, m1, m2), max3(m3, m4, KVC_F(15)));
#undef KVC_F
  const float m_new = fmaxf(m, cmax * scale);
  if (m_new > m) {
    const f32x2 corr = splat2(ex2(m - m_new));
    sum2[0] = mul2(sum2[0], corr);
    sum2[1] = mul2(sum2[1], corr);
    m = m_new;
  }
  const f32x2 nm = splat2(-m);
  sum2[0] = add2(sum2[0], exp2_mix2<0, KVC_POLY_PAIRS_LSE>(fma2(pack2(x[0], x[1]), scale2, nm)));
  sum2[1] = add2(sum2[1], exp2_mix2<1, KVC_POLY_PAIRS_LSE>(fma2(pack2(x[2], x[3]), scale2, nm)));
  sum2[0] = add2(sum2[0], exp2_mix2<2, KVC_POLY_PAIRS_LSE>(fma2(pack2(x[4], x[5]), scale2, nm)));
  sum2[1] = add2(sum2[1], exp2_mix2<3, KVC_POLY_PAIRS_LSE>(fma2(pack2(x[6], x[7]), scale2, nm)));
  sum2[0] = add2(sum2[0], exp2_mix2<4, KVC_POLY_PAIRS_LSE>(fma2(pack2(x[8], x[9]), scale2, nm)));
  sum2[1] = add2(sum2[1], exp2_mix2<5, KVC_POLY_PAIRS_LSE>(fma2(pack2(x[10], x[11]), scale2, nm)));
  sum2[0] = add2(sum2[0], exp2_mix2<6, KVC_POLY_PAIRS_LSE>(fma2(pack2(x[12], x[13]), scale2, nm)));
  sum2[1] = add2(sum2[1], exp2_mix2<7, KVC_POLY_PAIRS_LSE>(fma2(pack2(x[14], x[15]), scale2, nm)));
}
__device__ __forceinline__ float sum4(const f32x2 (&s)[2]) {
  float a, b, c, d;
  unpack2(s[0], a, b);
  unpack2(s[1], c, d);
  return (a + b) + (c + d);
}

// The same 16 columns added with the reference m left as it is (no maximum is taken): correct as long as no
// 2^(x - m) overflows.  The special-function unit returns +inf then, which the caller's range check sees in the
// sums; the polynomial path would wrap around instead, so the largest argument that went through it is tracked.
__device__ __forceinline__ void lse_piece_lazy(const uint32_t (&x)[16], f32x2 scale2, float m, f32x2 (&sum2)[2],
                                               float& poly_max) {
  const f32x2 nm = splat2(-m);
  auto term = [&](auto jc, uint32_t a, uint32_t b) {
    constexpr int J = decltype(jc)::value;
    constexpr bool poly = ((J % 8 + 1) * KVC_POLY_PAIRS_LSE) / 8 > ((J % 8) * KVC_POLY_PAIRS_LSE) / 8;
    const f32x2 arg = fma2(pack2(a, b), scale2, nm);
    if constexpr (poly) {
      float a0, a1;
      unpack2(arg, a0, a1);
      poly_max = max3(poly_max, a0, a1);
      return exp2_poly2(arg);
    } else {
      return exp2_sfu2(arg);
    }
  };
  sum2[0] = add2(sum2[0], term(std::integral_constant<int, 0>{}, x[0], x[1]));
  sum2[1] = add2(sum2[1], term(std::integral_constant<int, 1>{}, x[2], x[3]));
  sum2[0] = add2(sum2[0], term(std::integral_constant<int, 2>{}, x[4], x[5]));
  sum2[1] = add2(sum2[1], term(std::integral_constant<int, 3>{}, x[6], x[7]));
  sum2[0] = add2(sum2[0], term(std::integral_constant<int, 4>{}, x[8], x[9]));
  sum2[1] = add2(sum2[1], term(std::integral_constant<int, 5>{}, x[10], x[11]));
  sum2[0] = add2(sum2[0], term(std::integral_constant<int, 6>{}, x[12], x[13]));
  sum2[1] = add2(sum2[1], term(std::integral_constant<int, 7>{}, x[14], x[15]));
}

// Sweep 1, one whole accumulator (128 unmasked columns) for a row whose reference m is already finite.  The maximum
// of a softmax row rarely moves after its first tile, and the running sum may use any reference that keeps
// 2^(x - m) finite, so the first seven pieces are added against the reference as it stands, without the max tree.
// Before the accumulator is handed back the sums are checked: if any lane of the warp left the range, those pieces
// are redone exactly from TMEM; a sum that has grown past 2^60 moves the reference up by 60.  The last piece is
// already in registers and is added exactly.
template <class Release>
__device__ __forceinline__ void lse_tile_lazy(uint32_t taddr, float scale, f32x2 scale2, float& m, f32x2 (&sum2)[2],
                                              Release&& release) {
  uint32_t va[16], vb[16];
  const f32x2 keep0 = sum2[0], keep1 = sum2[1];
  float poly_max = 0.f;
  tmem_ld16(taddr, va);
  tmem_wait16(va);
#pragma unroll
  for (int p = 0; p < 6; p += 2) {
    tmem_ld16(taddr + (p + 1) * 16, vb);
    lse_piece_lazy(va, scale2, m, sum2, poly_max);
    tmem_wait16(vb);
    tmem_ld16(taddr + (p + 2) * 16, va);
    lse_piece_lazy(vb, scale2, m, sum2, poly_max);
    tmem_wait16(va);
  }
  tmem_ld16(taddr + 7 * 16, vb);
  lse_piece_lazy(va, scale2, m, sum2, poly_max);
  tmem_wait16(vb);
  const float total = sum4(sum2);
  if (__any_sync(0xFFFFFFFFu, !(total < 0x1p100f) || poly_max > 100.f)) {
    sum2[0] = keep0;
    sum2[1] = keep1;
#pragma unroll 1
    for (int p = 0; p < 7; ++p) {
      tmem_ld16(taddr + p * 16, va);
      tmem_wait16(va);
      lse_piece<false>(va, scale, scale2, 16, m, sum2);
    }
  } else if (total > 0x1p60f) {
    m += 60.f;
    const f32x2 down = splat2(0x1p-60f);
    sum2[0] = mul2(sum2[0], down);
    sum2[1] = mul2(sum2[1], down);
  }
  release();
  lse_piece<false>(vb, scale, scale2, 16, m, sum2);
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

// kind::f16 instruction descriptor: fp32 accumulate, both operands K-major and of one type (bf16 x bf16 or
// fp16 x fp16: format code 1 or 0 in the A and B fields), M x N.
__host__ __device__ constexpr uint32_t make_idesc(int m, int n, bool bf16) {
  return (1u << 4) | ((bf16 ? 1u : 0u) << 7) | ((bf16 ? 1u : 0u) << 10) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(m >> 4) << 24);
}


// ------------------------------------------------------------------------------------------------
// work decomposition: rank -> (sequence, tile), heaviest first
// ------------------------------------------------------------------------------------------------
// Items are (sequence, tile) pairs; an item's weight w is the number of 128x128 tiles it sweeps
// (causal: query tile q sweeps q+1 key tiles; key tile k sweeps n-k query tiles).  Rank j counts items
// in order of decreasing w, sequences in order inside one w.  Runs on one full warp.
// With an observation window (window > 0) a row sweep only has the items that hold one of the last
// `window` rows of their sequence; `tile` is then still the item's index inside the whole sequence.
__device__ __forceinline__ void decode_item(const int32_t* __restrict__ cu, int n_seqs, int max_tiles, int j,
                                            bool row_sweep, int lane, int& seq, int& tile, int& n_tiles,
                                            int rows_per_item, int window) {
  int rem = j;
  seq = 0; tile = 0; n_tiles = 0;
  if (n_seqs == 1) {                               // one sequence: rank j is simply the j-th heaviest item
    const int len = __ldg(cu + 1) - __ldg(cu);
    n_tiles = (len + rows_per_item - 1) / rows_per_item;
    tile = row_sweep ? n_tiles - 1 - j : j;
    return;
  }
  for (int w = max_tiles; w >= 1; --w) {
    for (int base = 0; base < n_seqs; base += 32) {
      const int s = base + lane;
      const int len = s < n_seqs ? __ldg(cu + s + 1) - __ldg(cu + s) : 0;
      const int nt = (len + rows_per_item - 1) / rows_per_item;
      const int first = (row_sweep && window > 0 && len > window) ? (len - window) / rows_per_item : 0;
      const int cnt_s = nt - first;
      const unsigned mask = __ballot_sync(0xFFFFFFFFu, cnt_s >= w);
      const int cnt = __popc(mask);
      if (rem < cnt) {
        const int pos = __fns(mask, 0, rem + 1);
        seq = base + pos;
        n_tiles = __shfl_sync(0xFFFFFFFFu, nt, pos);
        const int first_p = __shfl_sync(0xFFFFFFFFu, first, pos);
        tile = row_sweep ? first_p + w - 1 : n_tiles - w;
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

// 4-D view (channel, token, head, layer) of a token-major bf16 or fp16 tensor; box = 64 channels x 128 tokens.
// A stride only matters along an axis longer than 1; there it must be positive (the TMA unit cannot repeat a row)
// and inside the tensor map's 40-bit byte range.  Returns false for anything the map cannot describe.
inline bool make_map(CUtensorMap* map, const TensorView& t, int D, int T, int H, int n_layers) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  const cuuint64_t gdim[4] = {(cuuint64_t)D, (cuuint64_t)T, (cuuint64_t)H, (cuuint64_t)n_layers};
  const long long st[3] = {t.st, t.sh, t.sl};
  cuuint64_t gstride[3];
  for (int i = 0; i < 3; ++i) {
    if (gdim[i + 1] > 1) {
      if (st[i] <= 0 || st[i] >= (1LL << 38)) return false;
      gstride[i] = (cuuint64_t)st[i] * 2;
    } else {
      gstride[i] = 16;                                // never used to step: any legal value
    }
  }
  const cuuint32_t box[4] = {64, 128u, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return enc(map, t.dtype == KVCRUSH_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<void*>(t.ptr), gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


}  // namespace tc
}  // namespace kvc
