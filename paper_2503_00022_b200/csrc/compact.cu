// Stage 4: gather of the kept K/V rows into the reduced cache (Sec. 3.2 of the paper: the
// representatives together with the important tokens form the final cache).
//
// Pure byte movement, bound by HBM bandwidth.  One warp owns one kept token of one layer and
// copies that token's rows of every KV head, for K and for V, as 16-byte vectors: the index
// arithmetic (segment search, source token) is paid once per token, and every lane keeps four
// independent 16-byte loads in flight before the first store.
//
// Page-granular variant (Sec. 4.3.5: paged caches keep or drop whole pages): the kept list holds page numbers,
// a warp owns one token slot of one kept page, and the slots of a short last page are filled with zeros.
#include "common.cuh"

namespace kvc {

namespace {

constexpr int kWarpsPerBlock = 8;

struct CompactArgs {
  const unsigned char* src[2];
  unsigned char* dst[2];
  long long src_sl[2], src_st[2], src_sh[2];   // bytes
  long long dst_sl[2], dst_st[2], dst_sh[2];   // bytes
  int n_tensors;
  int vec_per_row;                             // 16-byte vectors in one head row
  int n_vec;                                   // vectors per token = Hkv * vec_per_row
};

template <bool kPaged>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
compact_kernel(Shape s, CompactArgs a, const int32_t* __restrict__ cu_kept, const int32_t* __restrict__ idx,
               long long total_kept, int page_size) {
  const int lane = threadIdx.x & 31;
  const long long out_row = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  // row = position in the kept list (a token, or a page of which this warp copies slot `slot`)
  const long long row = kPaged ? out_row / page_size : out_row;
  const int slot = kPaged ? (int)(out_row - row * page_size) : 0;
  if (row >= total_kept) return;

  // segment = layer * n_seqs + seq that owns kept row `row`
  const int n_seg = s.n_layers * s.n_seqs;
  int lo = 0, hi = n_seg;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if ((long long)__ldg(cu_kept + mid) <= row) lo = mid; else hi = mid;
  }
  const int layer = lo / s.n_seqs, seq = lo - layer * s.n_seqs;
  long long src_tok, dst_tok;
  bool present = true;
  if (kPaged) {
    const long long tok_in_seq = (long long)__ldg(idx + row) * page_size + slot;
    const int seq_begin = __ldg(s.cu_seqlens + seq);
    present = tok_in_seq < __ldg(s.cu_seqlens + seq + 1) - seq_begin;
    src_tok = seq_begin + tok_in_seq;
    dst_tok = (row - __ldg(cu_kept + layer * s.n_seqs)) * page_size + slot;
  } else {
    src_tok = (long long)__ldg(s.cu_seqlens + seq) + __ldg(idx + row);
    dst_tok = row - __ldg(cu_kept + layer * s.n_seqs);
  }

#pragma unroll 1
  for (int ten = 0; ten < a.n_tensors; ++ten) {
    const unsigned char* sp = a.src[ten] + layer * a.src_sl[ten] + src_tok * a.src_st[ten];
    unsigned char* dp = a.dst[ten] + layer * a.dst_sl[ten] + dst_tok * a.dst_st[ten];
    for (int v0 = lane; v0 < a.n_vec; v0 += 4 * 32) {
      uint4 val[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int v = v0 + u * 32;
        if (kPaged) val[u] = make_uint4(0u, 0u, 0u, 0u);
        if (v < a.n_vec && (!kPaged || present)) {
          const int h = v / a.vec_per_row, c = v - h * a.vec_per_row;
          val[u] = __ldcs(reinterpret_cast<const uint4*>(sp + h * a.src_sh[ten]) + c);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int v = v0 + u * 32;
        if (v < a.n_vec) {
          const int h = v / a.vec_per_row, c = v - h * a.vec_per_row;
          __stcs(reinterpret_cast<uint4*>(dp + h * a.dst_sh[ten]) + c, val[u]);
        }
      }
    }
  }
}

}  // namespace

namespace {

// Running scores follow the cache: out[l][h][dst] = in[l][h][src] for the kept tokens (or the slots of the kept
// pages; slots past the end of a sequence get 0).  One thread per (layer, kept row), looping over the heads.
__global__ void __launch_bounds__(256)
compact_scores_kernel(Shape s, const float* __restrict__ in, float* __restrict__ out, const int32_t* __restrict__ cu_kept,
                      const int32_t* __restrict__ idx, long long total_kept, int page_size, long long out_tokens) {
  const long long out_row = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long row = out_row / page_size;
  const int slot = (int)(out_row - row * page_size);
  if (row >= total_kept) return;
  const int n_seg = s.n_layers * s.n_seqs;
  int lo = 0, hi = n_seg;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if ((long long)__ldg(cu_kept + mid) <= row) lo = mid; else hi = mid;
  }
  const int layer = lo / s.n_seqs, seq = lo - layer * s.n_seqs;
  const int seq_begin = __ldg(s.cu_seqlens + seq);
  const long long tok_in_seq = (long long)__ldg(idx + row) * page_size + slot;
  const bool present = tok_in_seq < __ldg(s.cu_seqlens + seq + 1) - seq_begin;
  const long long dst = (row - __ldg(cu_kept + layer * s.n_seqs)) * page_size + slot;
  const float* src = in + (long long)layer * s.Hq * s.T + seq_begin + tok_in_seq;
  float* dp = out + (long long)layer * s.Hq * out_tokens + dst;
  for (int h = 0; h < s.Hq; ++h) dp[(long long)h * out_tokens] = present ? __ldg(src + (long long)h * s.T) : 0.f;
}

int launch_gather(const Shape& s, const TensorView& K, const TensorView* V, int page_size, const int32_t* cu_kept,
                  const int32_t* idx, long long total_kept, const TensorView& K_out, const TensorView* V_out,
                  cudaStream_t stream) {
  if (total_kept == 0) return KVCRUSH_OK;
  const int eb = elt_bytes(K.dtype);
  CompactArgs a{};
  a.n_tensors = V ? 2 : 1;
  const TensorView* in[2] = {&K, V};
  const TensorView* out[2] = {&K_out, V_out};
  for (int i = 0; i < a.n_tensors; ++i) {
    a.src[i] = static_cast<const unsigned char*>(in[i]->ptr);
    a.dst[i] = static_cast<unsigned char*>(const_cast<void*>(out[i]->ptr));
    a.src_sl[i] = in[i]->sl * eb; a.src_st[i] = in[i]->st * eb; a.src_sh[i] = in[i]->sh * eb;
    a.dst_sl[i] = out[i]->sl * eb; a.dst_st[i] = out[i]->st * eb; a.dst_sh[i] = out[i]->sh * eb;
  }
  a.vec_per_row = s.D * eb / 16;
  a.n_vec = s.Hkv * a.vec_per_row;
  const long long rows = total_kept * (page_size > 0 ? page_size : 1);
  const long long blocks = (rows + kWarpsPerBlock - 1) / kWarpsPerBlock;
  if (blocks > 0x7FFFFFFFLL) return KVCRUSH_ERR_UNSUPPORTED;
  if (page_size > 0)
    compact_kernel<true><<<(unsigned)blocks, kWarpsPerBlock * 32, 0, stream>>>(s, a, cu_kept, idx, total_kept, page_size);
  else
    compact_kernel<false><<<(unsigned)blocks, kWarpsPerBlock * 32, 0, stream>>>(s, a, cu_kept, idx, total_kept, 1);
  return check_launch();
}

}  // namespace

int launch_compact(const Shape& s, const TensorView& K, const TensorView* V, const int32_t* cu_kept,
                   const int32_t* idx, long long total_kept, const TensorView& K_out, const TensorView* V_out,
                   cudaStream_t stream) {
  return launch_gather(s, K, V, 0, cu_kept, idx, total_kept, K_out, V_out, stream);
}

int launch_compact_scores(const Shape& s, const float* scores_in, int page_size, const int32_t* cu_kept,
                          const int32_t* idx, long long total_kept, float* scores_out, long long out_tokens,
                          cudaStream_t stream) {
  if (total_kept == 0) return KVCRUSH_OK;
  const int ps = page_size > 0 ? page_size : 1;
  const long long rows = total_kept * ps;
  const long long blocks = (rows + 255) / 256;
  if (blocks > 0x7FFFFFFFLL) return KVCRUSH_ERR_UNSUPPORTED;
  compact_scores_kernel<<<(unsigned)blocks, 256, 0, stream>>>(s, scores_in, scores_out, cu_kept, idx, total_kept, ps,
                                                             out_tokens);
  return check_launch();
}

int launch_compact_pages(const Shape& s, const TensorView& K, const TensorView* V, int page_size,
                         const int32_t* cu_kept, const int32_t* page_idx, long long total_kept_pages,
                         const TensorView& K_out, const TensorView* V_out, cudaStream_t stream) {
  return launch_gather(s, K, V, page_size, cu_kept, page_idx, total_kept_pages, K_out, V_out, stream);
}

}  // namespace kvc
