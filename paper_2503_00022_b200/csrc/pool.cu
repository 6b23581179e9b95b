// Max pooling of the per-head scores along the token axis (SnapKV's way of keeping the neighbours of a
// high-scoring token, named in Sec. 2.3 / 4.1.1 of the paper): out[l][h][t] = max over the centred window of
// odd width `kernel`, clipped to t's own sequence.  One thread per output; lanes are consecutive tokens, so
// the window reads of a warp overlap and come from L1.
#include "common.cuh"

namespace kvc {

namespace {

__global__ void __launch_bounds__(256)
pool_scores_kernel(Shape s, const float* __restrict__ in, int radius, float* __restrict__ out) {
  const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long n = (long long)s.n_layers * s.Hq * s.T;
  if (gid >= n) return;
  const int tok = (int)(gid % s.T);
  const int seq = seq_of_token(s.cu_seqlens, s.n_seqs, tok);
  const int lo = max(__ldg(s.cu_seqlens + seq), tok - radius);
  const int hi = min(__ldg(s.cu_seqlens + seq + 1) - 1, tok + radius);
  const float* row = in + (gid - tok);
  float m = __ldg(row + lo);
  for (int t = lo + 1; t <= hi; ++t) m = fmaxf(m, __ldg(row + t));
  out[gid] = m;
}

}  // namespace

int launch_pool_scores(const Shape& s, const float* scores_in, int kernel, float* scores_out, cudaStream_t stream) {
  const long long n = (long long)s.n_layers * s.Hq * s.T;
  if (n == 0) return KVCRUSH_OK;
  const long long blocks = (n + 255) / 256;
  if (blocks > 0x7FFFFFFFLL) return KVCRUSH_ERR_UNSUPPORTED;
  pool_scores_kernel<<<(unsigned)blocks, 256, 0, stream>>>(s, scores_in, (kernel - 1) / 2, scores_out);
  return check_launch();
}

}  // namespace kvc
