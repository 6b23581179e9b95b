// Shared declarations of the kvcrush CUDA library (internal; the public ABI is include/kvcrush.h).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "kvcrush.h"

namespace kvc {

// Device-side view of the problem shape, passed by value to every kernel.
struct Shape {
  int n_layers, n_seqs, Hq, Hkv, D, T, max_seqlen, causal;
  int G;                       // Hq / Hkv
  int W;                       // signature words per token
  int window;                  // > 0: only the last `window` queries of each sequence vote (observation window)
  const int32_t* cu_seqlens;   // device, [n_seqs + 1]
};

struct TensorView {
  const void* ptr;
  int dtype;
  long long sl, st, sh;        // strides in elements: layer, token, head
};

inline int elt_bytes(int dtype) { return dtype == KVCRUSH_FP32 ? 4 : 2; }

// kernel ids written to status[1]
enum KernelId { KID_SCORE_LSE = 1, KID_SCORE_COLSUM = 2, KID_KMEANS = 3 };

__device__ __forceinline__ void report(int32_t* status, int code, int kid, int a, int b) {
  if (atomicCAS(status, 0, code) == 0) {
    status[1] = kid;
    status[2] = a;
    status[3] = b;
  }
}

// Sequence that owns packed token `tok` (binary search in cu_seqlens).
__device__ __forceinline__ int seq_of_token(const int32_t* __restrict__ cu, int n_seqs, int tok) {
  int lo = 0, hi = n_seqs;          // invariant: cu[lo] <= tok < cu[hi]
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (__ldg(cu + mid) <= tok) lo = mid; else hi = mid;
  }
  return lo;
}

// ---- stage launchers (defined in the per-stage .cu files) -------------------------------------------

// score: SIMT fp32 kernels (any dtype/shape) and tcgen05 kernels (bf16 or fp16, D a multiple of 8 up to 128).
// lse2_ws: [n_layers][Hq][T] float32 row log-sum-exp in the log2 domain (written unless lse_in is given).
int launch_score_simt(const Shape& s, const TensorView& Q, const TensorView& K, float scale_log2,
                      const float* lse_in, float lse_in_mul, float* lse2_ws, float* scores, float* lse_out,
                      int normalize, int32_t* status, cudaStream_t stream);
// Decode step: scores[l][h][t] += attention of sequence(t)'s new query (Q_new's token axis = sequence) to key t.
int launch_score_decode(const Shape& s, const TensorView& Q_new, const TensorView& K, float scale_log2, float* scores,
                        cudaStream_t stream);
// Can the tensor-core kernels take this problem?  On TENSOR_PLAN_OK `maps` holds the two encoded tensor maps.
enum { TENSOR_PLAN_OK = 0,
       TENSOR_PLAN_NO = 1,            // type, head_dim or strides outside what the kernels / the TMA unit take
       TENSOR_PLAN_NO_ENCODER = 2 };  // the problem qualifies but the driver has no tensor-map encoder
struct ScoreTensorMaps { alignas(64) unsigned char q[128]; alignas(64) unsigned char k[128]; };   // two CUtensorMap
int score_tensor_plan(const Shape& s, const TensorView& Q, const TensorView& K, ScoreTensorMaps* maps);
// Diagnostics of one launch (all zero in normal use).
struct ScoreDiag {
  int short_waits;           // run the kernels instantiated with a short limit on every bounded barrier wait
  int withhold_first_item;   // the producer warp of every CTA stops before announcing its first work item
};
// `counters`: two ints of caller scratch (work counters of the two persistent sweeps).
size_t score_tensor_counter_bytes();
int launch_score_tensor(const Shape& s, const int32_t* cu_host, const TensorView& Q, const ScoreTensorMaps& maps,
                        float scale_log2, const float* lse_in, float lse_in_mul, float* lse2_ws, int* counters,
                        float* scores, float* lse_out, int normalize, int32_t* status, const ScoreDiag& diag,
                        cudaStream_t stream);

// importance: optional out [n_layers][T] float64, the token importance I(t) of stage 3 (written from the same loads).
int launch_signature(const Shape& s, const float* scores, const int32_t* sig_keep, const float* theta_in,
                     uint32_t* sigs, float* theta, double* importance, cudaStream_t stream);

size_t select_workspace_bytes(const Shape& s);
// importance: optional [n_layers][T] float64 I(t) from the signature stage; NULL: computed from the scores.
int launch_select(const Shape& s, const float* scores, const double* importance, const uint32_t* sigs,
                  const int32_t* budget_imp,
                  const int32_t* budget_rep, int anchor_mode, const uint32_t* anchor_bits, int anchor_per_segment,
                  int keep_initial, int keep_recent, const int32_t* cu_kept, int32_t* idx, uint8_t* kind,
                  int32_t* n_kept, void* ws, cudaStream_t stream);

// Order-preserving 64-bit keys of the token importance I(t), [n_layers][T] (first kernel of the selection stages).
int launch_importance(const Shape& s, const float* scores, int keep_initial, int keep_recent,
                      unsigned long long* keys, cudaStream_t stream);

// The same keys from an importance array [n_layers][T] the caller supplies.
int launch_importance_keys(const Shape& s, const double* importance, int keep_initial, int keep_recent,
                           unsigned long long* keys, cudaStream_t stream);

// Clustering baseline (k-means in the place of Algorithm 2's grouping); max_budget_rep bounds every budget_rep.
size_t kmeans_workspace_bytes(const Shape& s, int max_budget_rep);
bool kmeans_supported(const Shape& s);
int launch_kmeans_select(const Shape& s, const float* scores, const double* importance, const uint32_t* sigs,
                         const int32_t* budget_imp, const int32_t* budget_rep, int max_budget_rep, int iterations,
                         int keep_initial, int keep_recent, const int32_t* cu_kept, int32_t* idx, uint8_t* kind,
                         int32_t* n_kept, void* ws, int32_t* status, cudaStream_t stream);

// Page-granular selection and gather (a page = page_size consecutive tokens of one sequence).
constexpr int kMaxPagesPerSeq = 8192;      // pages of one sequence the page kernel holds in shared memory
constexpr int kMaxPageWords = 128;         // signature words of one page (page_size * W)
int launch_select_pages(const Shape& s, const float* scores, const double* importance, const uint32_t* sigs,
                        int page_size,
                        const int32_t* budget_imp, const int32_t* budget_rep, int anchor_mode,
                        const uint32_t* anchor_bits, int anchor_per_segment, int keep_initial, int keep_recent,
                        const int32_t* cu_kept, int32_t* page_idx, uint8_t* kind, int32_t* n_kept, void* ws,
                        cudaStream_t stream);
int launch_compact_pages(const Shape& s, const TensorView& K, const TensorView* V, int page_size,
                         const int32_t* cu_kept, const int32_t* page_idx, long long total_kept_pages,
                         const TensorView& K_out, const TensorView* V_out, cudaStream_t stream);

// Gather of the running scores along the kept tokens (page_size 0) or kept pages.
int launch_compact_scores(const Shape& s, const float* scores_in, int page_size, const int32_t* cu_kept,
                          const int32_t* idx, long long total_kept, float* scores_out, long long out_tokens,
                          cudaStream_t stream);

int launch_pool_scores(const Shape& s, const float* scores_in, int kernel, float* scores_out, cudaStream_t stream);

int launch_compact(const Shape& s, const TensorView& K, const TensorView* V, const int32_t* cu_kept,
                   const int32_t* idx, long long total_kept, const TensorView& K_out, const TensorView* V_out,
                   cudaStream_t stream);

// Validates a problem description and fills the device-side view (defined in api.cu).
int shape_from_problem(const kvcrush_problem_t* problem, Shape* out);

inline int check_launch() { return cudaGetLastError() == cudaSuccess ? KVCRUSH_OK : KVCRUSH_ERR_CUDA; }

}  // namespace kvc
